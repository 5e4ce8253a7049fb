"""The multi-process side of the path on CPU (gloo, world size 2): sequences are sharded with
no overlap, each rank regenerates the permutations of its own sequences from (seed, layer, b),
and the only cross-rank reduction -- the gate-logit gradient -- matches the full-batch value.
The per-rank arithmetic is the float64 oracle; the CUDA path is not involved."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2604_00754_b200.dist import allreduce_gate_grads, shard_range

B, HQ, HKV, N, D, W, SEED, LAYER = 5, 4, 2, 48, 8, 9, 21, 3
FLAGS = 1 | 4


def inputs():
    g = np.random.default_rng(7)
    q = g.standard_normal((B, HQ, N, D)); k = g.standard_normal((B, HKV, N, D))
    v = g.standard_normal((B, HKV, N, D)); dy = g.standard_normal((B, HQ, N, D))
    lg = g.standard_normal((2, HQ))
    return q, k, v, dy, lg


def worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, k, v, dy, lg = inputs()
    lo, hi = shard_range(B, rank, world)
    # permutations of the owned sequences only: sequence b must come out the same as in a
    # full-batch call, whatever the rank that draws it
    full_perm, full_inv = oracle.make_perm(SEED, LAYER, B, N)
    perm = np.stack([oracle.make_perm(SEED, LAYER, b + 1, N)[0][b] for b in range(lo, hi)])
    assert np.array_equal(perm, full_perm[lo:hi])
    dq, dk, dv, dg = oracle.backward(q[lo:hi], k[lo:hi], v[lo:hi], full_perm[lo:hi],
                                     full_inv[lo:hi], lg, dy[lo:hi], W, FLAGS)
    dgt = torch.from_numpy(np.ascontiguousarray(dg))
    allreduce_gate_grads(dgt)
    owned = torch.zeros(B, dtype=torch.int64)
    owned[lo:hi] = 1
    dist.all_reduce(owned)
    if rank == 0:
        out["dgate"] = dgt.numpy().copy()
        out["owned"] = owned.numpy().copy()
        out["dq0"] = dq[0].copy()
    dist.destroy_process_group()


def test_batch_shards_and_gate_gradient_allreduce():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(worker, args=(2, port, out), nprocs=2, join=True)
    assert list(out["owned"]) == [1] * B                     # every sequence exactly once
    q, k, v, dy, lg = inputs()
    perm, inv = oracle.make_perm(SEED, LAYER, B, N)
    dq, _, _, dg = oracle.backward(q, k, v, perm, inv, lg, dy, W, FLAGS)
    assert np.allclose(out["dgate"], dg, rtol=1e-12, atol=1e-12)
    assert np.array_equal(out["dq0"], dq[0])                 # per-sequence results do not mix


def test_shard_range_partitions():
    for Bn in (1, 2, 5, 8, 13):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                lo, hi = shard_range(Bn, r, world)
                seen += list(range(lo, hi))
            assert seen == list(range(Bn))
