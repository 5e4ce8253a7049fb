// Gated combination of the two branch outputs (Eq. 5, per-head scalar gates) as a streaming
// kernel: y = sigmoid(logit[0,h]) * y_sa + sigmoid(logit[1,h]) * y_swa.  One thread moves
// 16 bytes of each tensor; y may be one of the inputs (every element is read and written by
// the same thread).  HBM-bound: two rows in, one row out per (token, head).
#include "sa_common.cuh"

namespace sa {
namespace {

template <typename T> struct Vec;
template <> struct Vec<float> { static constexpr int kN = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int kN = 8; };

template <typename T>
__global__ void combine_kernel(T* __restrict__ y, const T* y_sa, const T* y_swa,
                               const float* __restrict__ logits, int Hq, int n, int d,
                               int64_t s0, int64_t s1, int64_t s2, int64_t total) {
  constexpr int V = Vec<T>::kN;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int per_row = d / V;
  const int64_t r = idx / per_row;
  const int c = (int)(idx - r * per_row) * V;
  const int tok = (int)(r % n);
  const int64_t bh = r / n;
  const int h = (int)(bh % Hq);
  const int64_t off = (bh / Hq) * s0 + h * s1 + (int64_t)tok * s2 + c;
  const float g_sa = 1.f / (1.f + __expf(-logits[h]));
  const float g_swa = 1.f / (1.f + __expf(-logits[Hq + h]));
  const uint4 a = *reinterpret_cast<const uint4*>(y_sa + off);
  const uint4 b = *reinterpret_cast<const uint4*>(y_swa + off);
  uint4 o;
  if (sizeof(T) == 4) {
    const float* fa = reinterpret_cast<const float*>(&a);
    const float* fb = reinterpret_cast<const float*>(&b);
    float* fo = reinterpret_cast<float*>(&o);
#pragma unroll
    for (int x = 0; x < 4; ++x) fo[x] = fmaf(g_swa, fb[x], g_sa * fa[x]);
  } else {
    const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b);
    __nv_bfloat162* ho = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int x = 0; x < 4; ++x)
      ho[x] = __floats2bfloat162_rn(fmaf(g_swa, __low2float(hb[x]), g_sa * __low2float(ha[x])),
                                    fmaf(g_swa, __high2float(hb[x]), g_sa * __high2float(ha[x])));
  }
  *reinterpret_cast<uint4*>(y + off) = o;
}

}  // namespace

cudaError_t launch_combine(void* y, const void* y_sa, const void* y_swa, const float* logits,
                           int B, int Hq, int n, int d, const int64_t s[3], int dtype,
                           cudaStream_t st) {
  const int V = dtype == SA_BF16 ? 8 : 4;
  const int64_t total = (int64_t)B * Hq * n * (d / V);
  const int64_t blocks = (total + 255) / 256;
  if (blocks > 0x7fffffffll) return cudaErrorInvalidValue;
  if (dtype == SA_BF16)
    combine_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(
        (__nv_bfloat16*)y, (const __nv_bfloat16*)y_sa, (const __nv_bfloat16*)y_swa, logits, Hq, n,
        d, s[0], s[1], s[2], total);
  else
    combine_kernel<float><<<(unsigned)blocks, 256, 0, st>>>((float*)y, (const float*)y_sa,
                                                            (const float*)y_swa, logits, Hq, n, d,
                                                            s[0], s[1], s[2], total);
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa
