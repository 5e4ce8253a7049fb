"""Stochastic Attention hot path for B200 (sm_100a): thin Python binding over a C-ABI CUDA library."""
