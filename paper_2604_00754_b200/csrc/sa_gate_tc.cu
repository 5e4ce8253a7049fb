// Projection gates of Eq. 5-6 for sm_100a: out = sigmoid(Y_sa W_sa^T) * Y_sa
// (+ sigmoid(Y_swa W_swa^T) * Y_swa), the attention block's last step before its output
// projection (App. B).
//
// A dense contraction, so it runs on the 5th-generation tensor cores: a persistent grid of
// one CTA per SM walks 128 x 128 output tiles.  Warp 0 streams 128 x 64 tiles of Y and of W
// (both K-major, 128-byte swizzle) through a three-stage ring with TMA, warp 1 issues
// tcgen05.mma into two fp32 accumulators per tile (one per path) in tensor memory, warps 2-9
// read a finished pair of accumulators, apply the logistic, multiply by the rows of Y and
// write the tile while the next tile's products already run into the other pair.  Tiles are
// visited in blocks of 16 column tiles so that the slice of W in use stays in L2.
//
// Every mbarrier wait is bounded; on expiry the CTA records SA_ERR_TIMEOUT in the device
// status word, stops issuing work, drains what it started and returns.
#include "sa_gemm_common.cuh"

namespace sa {
namespace {

constexpr int kBM = 128, kBN = 128, kBK = 64;
constexpr int kStages = 3;
constexpr int kTileBytes = 128 * kBK * 2;             // one 128 x 64 bf16 tile
// a stage: Y_sa, W_sa, Y_swa, W_swa of one 64-wide K chunk, or, for the single path, Y, W of
// two consecutive K chunks (so that one hand-over always feeds eight products)
constexpr int kStageBytes = 4 * kTileBytes;
constexpr int kGateThreads = 320;                    // TMA, MMA and eight epilogue warps
constexpr int kOffBars = kStages * kStageBytes;
// barriers: full[kStages], empty[kStages], acc_full[2], acc_empty[2]
constexpr int kBarFull = 0, kBarEmpty = kStages, kBarAccFull = 2 * kStages,
              kBarAccEmpty = 2 * kStages + 2, kNumBars = 2 * kStages + 4;
constexpr int kOffMisc = kOffBars + kNumBars * 8;     // TMEM base address, gave_up flag
constexpr int kGateSmem = kOffMisc + 16;

struct GateParams {
  const __nv_bfloat16 *y_sa, *y_swa;
  __nv_bfloat16* out;
  int64_t rows, ld_y, ld_out;
  int dm, dual;
  int tiles_m, tiles_n, k_chunks;
  int* status;
};

// Tile order: blocks of kNB column tiles, inside a block row tile by row tile.  The CTAs that
// run at the same time then share a slice of W that stays in L2 (kNB x 1 MB per path at
// dm = 4096) while Y streams through once per block.
constexpr int kNB = 16;
__device__ __forceinline__ void tile_origin(const GateParams& p, int tile, int* m0, int* n0) {
  const int per_block = p.tiles_m * kNB;
  const int nb = tile / per_block, rem = tile - nb * per_block;
  const int width = min(kNB, p.tiles_n - nb * kNB);
  *m0 = (rem / width) * kBM;
  *n0 = (nb * kNB + rem % width) * kBN;
}

__global__ void __launch_bounds__(kGateThreads, 1)
gate_tc_kernel(const __grid_constant__ GateParams p, const __grid_constant__ CUtensorMap tm_ysa,
               const __grid_constant__ CUtensorMap tm_wsa, const __grid_constant__ CUtensorMap tm_yswa,
               const __grid_constant__ CUtensorMap tm_wswa) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                        // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) atomicCAS(p.status, SA_OK, SA_ERR_CUDA);
    return;
  }
  const uint32_t bar0 = sbase + kOffBars;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc);
  volatile int* gave_up = reinterpret_cast<volatile int*>(smem + kOffMisc + 4);

  if (threadIdx.x == 0) {
    *gave_up = 0;
    note_skip(reinterpret_cast<volatile int*>(smem + kOffMisc + 8), p.status, nullptr);
    for (int i = 0; i < kNumBars; ++i)
      mbar_init(bar(i), (i >= kBarAccEmpty) ? 256 : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  SA_LEAVE_IF_SKIPPED(reinterpret_cast<volatile int*>(smem + kOffMisc + 8), 1, tmem, 512u)
  const int total = p.tiles_m * p.tiles_n;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t use = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        int m0, n0;
        tile_origin(p, tile, &m0, &n0);
        for (int kc = 0; kc < p.k_chunks && ok; ++kc, ++use) {
          const uint32_t s = use % kStages;
          if (use >= (uint32_t)kStages)
            ok = mbar_wait(bar(kBarEmpty + s), (use / kStages - 1) & 1u, gave_up, p.status);
          if (!ok) break;
          const uint32_t dst = sbase + s * kStageBytes, fb = bar(kBarFull + s);
          mbar_expect_tx(fb, kStageBytes);
          // single path: the second pair is the next K chunk (zeros past the last one)
          const int k0 = (p.dual ? kc : 2 * kc) * kBK, k1 = p.dual ? k0 : k0 + kBK;
          tma_load_2d(dst, &tm_ysa, k0, m0, fb);
          tma_load_2d(dst + kTileBytes, &tm_wsa, k0, n0, fb);
          tma_load_2d(dst + 2 * kTileBytes, &tm_yswa, k1, m0, fb);
          tma_load_2d(dst + 3 * kTileBytes, &tm_wswa, k1, n0, fb);
        }
      }
      // Loads that were started but never consumed (only after a failed wait) must land
      // before the shared memory goes away: wait for them, again with a limit.
      if (!ok || *gave_up) {
        const uint32_t first = use > (uint32_t)kStages ? use - kStages : 0u;
        for (uint32_t u = first; u < use; ++u)
          for (int tries = 0; tries < 100000; ++tries) {
            if (mbar_try(bar(kBarFull + u % kStages), (u / kStages) & 1u)) break;
            __nanosleep(100);
          }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kBM, kBN, false);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t kLoK = (16u >> 4) << 16;
      uint32_t use = 0, it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++it) {
        const uint32_t buf = it & 1u;
        if (it >= 2)   // the epilogue has read this pair of accumulators
          ok = mbar_wait(bar(kBarAccEmpty + buf), (it / 2 - 1) & 1u, gave_up, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_sa = tmem + buf * 256, d_swa = d_sa + 128;
        for (int kc = 0; kc < p.k_chunks && ok; ++kc, ++use) {
          const uint32_t s = use % kStages;
          ok = mbar_wait(bar(kBarFull + s), (use / kStages) & 1u, gave_up, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t lo = (sbase + s * kStageBytes) >> 4;
          mma_ss_x4(d_sa, desc64(lo | kLoK, kDescHi), desc64((lo + (kTileBytes >> 4)) | kLoK, kDescHi),
                    idesc, kc > 0);
          mma_ss_x4(p.dual ? d_swa : d_sa, desc64((lo + 2 * (kTileBytes >> 4)) | kLoK, kDescHi),
                    desc64((lo + 3 * (kTileBytes >> 4)) | kLoK, kDescHi), idesc,
                    p.dual ? (uint32_t)(kc > 0) : 1u);
          tc_commit(bar(kBarEmpty + s));      // the stage is free once these products are done
        }
        if (ok) tc_commit(bar(kBarAccFull + buf));
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------- epilogue (warps 2-9)
    // A warp reads the 32 TMEM lanes 32 (warp % 4) .. +31: one output row per thread, and
    // warps 2-5 take the first 64 columns of the tile, warps 6-9 the other 64.
    const int half = (warp - 2) >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
      const uint32_t buf = it & 1u;
      int m0, n0;
      tile_origin(p, tile, &m0, &n0);
      ok = mbar_wait(bar(kBarAccFull + buf), (it / 2) & 1u, gave_up, p.status);
      ok = __all_sync(0xffffffffu, ok);       // the tensor-memory loads are warp-collective
      if (!ok) break;
      tc_fence_after();
      const int64_t r = (int64_t)m0 + row;
      const bool row_ok = r < p.rows;
      const __nv_bfloat16* ya = p.y_sa + r * p.ld_y + n0;
      const __nv_bfloat16* yb = p.dual ? p.y_swa + r * p.ld_y + n0 : nullptr;
      __nv_bfloat16* o = p.out + r * p.ld_out + n0;
#pragma unroll 1
      for (int c = 2 * half; c < 2 * half + 2; ++c) {
        // the rows of Y are requested together, ahead of the stores they may not pass (out may
        // alias them as far as the compiler knows), so that their latencies overlap
        uint4 fa[4], fb[4];
        if (row_ok && n0 + 32 * c < p.dm) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            fa[x8] = *reinterpret_cast<const uint4*>(ya + 32 * c + 8 * x8);
            if (p.dual) fb[x8] = *reinterpret_cast<const uint4*>(yb + 32 * c + 8 * x8);
          }
        }
        uint32_t za[32], zb[32];
        tmem_ld32(tmem + lane_addr + buf * 256 + 32 * c, za);
        if (p.dual) tmem_ld32(tmem + lane_addr + buf * 256 + 128 + 32 * c, zb);
        tmem_wait_ld();
        if (row_ok && n0 + 32 * c < p.dm) {       // dm is a multiple of 64: whole chunks only
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&fa[x8]);
            float r8[8];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              r8[2 * x] = logistic(__uint_as_float(za[8 * x8 + 2 * x])) * __low2float(ha[x]);
              r8[2 * x + 1] = logistic(__uint_as_float(za[8 * x8 + 2 * x + 1])) * __high2float(ha[x]);
            }
            if (p.dual) {
              const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&fb[x8]);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                r8[2 * x] = fmaf(logistic(__uint_as_float(zb[8 * x8 + 2 * x])), __low2float(hb[x]),
                                 r8[2 * x]);
                r8[2 * x + 1] = fmaf(logistic(__uint_as_float(zb[8 * x8 + 2 * x + 1])),
                                     __high2float(hb[x]), r8[2 * x + 1]);
              }
            }
            uint4 st;
            __nv_bfloat162* hs = reinterpret_cast<__nv_bfloat162*>(&st);
#pragma unroll
            for (int x = 0; x < 4; ++x) hs[x] = __floats2bfloat162_rn(r8[2 * x], r8[2 * x + 1]);
            *reinterpret_cast<uint4*>(o + 32 * c + 8 * x8) = st;
          }
        }
      }
      // the accumulators may be overwritten once every thread of the eight warps has read them
      tc_fence_before();
      mbar_arrive(bar(kBarAccEmpty + buf));
    }
  }

  // ----------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u)
                 : "memory");
  }
}

// Plain kernel for everything the tensor-core path does not take (fp32, dm not a multiple of
// 64, unaligned rows): one thread per output element, fp32 accumulation.
template <typename T>
__global__ void gate_simt_kernel(int64_t rows, int dm, const T* __restrict__ y_sa,
                                 const T* __restrict__ y_swa, int64_t ld_y,
                                 const T* __restrict__ w_sa, const T* __restrict__ w_swa,
                                 T* __restrict__ out, int64_t ld_out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * dm) return;
  const int64_t r = idx / dm;
  const int o = (int)(idx % dm);
  float acc = 0.f;
  {
    const T* y = y_sa + r * ld_y;
    const T* w = w_sa + (int64_t)o * dm;
    float z = 0.f;
    for (int i = 0; i < dm; ++i) z = fmaf(to_f32(y[i]), to_f32(w[i]), z);
    acc = to_f32(y[o]) / (1.f + expf(-z));
  }
  if (y_swa) {
    const T* y = y_swa + r * ld_y;
    const T* w = w_swa + (int64_t)o * dm;
    float z = 0.f;
    for (int i = 0; i < dm; ++i) z = fmaf(to_f32(y[i]), to_f32(w[i]), z);
    acc += to_f32(y[o]) / (1.f + expf(-z));
  }
  out[r * ld_out + o] = from_f32<T>(acc);
}

}  // namespace
}  // namespace sa

extern "C" sa_status sa_gate_projection_forward(int64_t rows, int32_t dm, int32_t dtype,
                                                const void* y_sa, const void* y_swa, int64_t ld_y,
                                                const void* w_sa, const void* w_swa, void* out,
                                                int64_t ld_out, sa_stream_t stream) {
  using namespace sa;
  if (rows < 1 || dm < 1 || ld_y < dm || ld_out < dm || !y_sa || !w_sa || !out) return SA_ERR_INVALID_ARG;
  if (y_swa && !w_swa) return SA_ERR_INVALID_ARG;
  if (dtype != SA_F32 && dtype != SA_BF16) return SA_ERR_INVALID_ARG;
  if (rows * (int64_t)dm > (1ll << 40)) return SA_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc_off = debug_option(SA_DEBUG_TENSOR_CORES) == 0;
  const bool tc = !tc_off && dtype == SA_BF16 && dm % 64 == 0 && ld_y % 8 == 0 && ld_out % 8 == 0 &&
                  aligned16(y_sa) && aligned16(w_sa) && aligned16(out) &&
                  (!y_swa || (aligned16(y_swa) && aligned16(w_swa))) &&
                  rows < (1ll << 31) - 128;
  // Large products run one 128 x 256-tile launch per path (a quarter fewer operand bytes per
  // flop; the second path adds to the rounded result of the first); the fused dual-accumulator
  // kernel below serves the rest, and everything after
  // sa_debug_set(SA_DEBUG_GATE_WIDE_TILES, 0).
  const bool wide_on = debug_option(SA_DEBUG_GATE_WIDE_TILES) != 0;
  if (tc && wide_on) {
    int dev = 0, sms = 0;
    int* status = status_ptr();
    if (!status || cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return SA_ERR_CUDA;
    cudaError_t err;
    if (gate_forward_wide(rows, dm, y_sa, y_swa, ld_y, w_sa, w_swa, out, ld_out, status, sms, st,
                          &err))
      return err == cudaSuccess ? SA_OK : SA_ERR_CUDA;
  }
  if (tc) {
    CUtensorMap tm[4];
    const void* ysw = y_swa ? y_swa : y_sa;      // unused maps still have to be valid
    const void* wsw = y_swa ? w_swa : w_sa;
    if (!make_map(&tm[0], y_sa, rows, dm, ld_y, 128) || !make_map(&tm[1], w_sa, dm, dm, dm, 128) ||
        !make_map(&tm[2], ysw, rows, dm, ld_y, 128) || !make_map(&tm[3], wsw, dm, dm, dm, 128))
      return SA_ERR_CUDA;
    GateParams p{};
    p.y_sa = (const __nv_bfloat16*)y_sa;
    p.y_swa = (const __nv_bfloat16*)y_swa;
    p.out = (__nv_bfloat16*)out;
    p.rows = rows; p.ld_y = ld_y; p.ld_out = ld_out;
    p.dm = dm; p.dual = y_swa != nullptr;
    p.tiles_m = (int)((rows + kBM - 1) / kBM);
    p.tiles_n = (dm + kBN - 1) / kBN;
    p.k_chunks = p.dual ? dm / kBK : (dm / kBK + 1) / 2;    // hand-overs per tile
    p.status = status_ptr();
    if (!p.status) return SA_ERR_CUDA;
    if ((int64_t)p.tiles_m * p.tiles_n > 0x3fffffff) return SA_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return SA_ERR_CUDA;
    if (cudaFuncSetAttribute(gate_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kGateSmem) != cudaSuccess)
      return SA_ERR_CUDA;
    const int total = p.tiles_m * p.tiles_n;
    gate_tc_kernel<<<min(total, sms), kGateThreads, kGateSmem, st>>>(p, tm[0], tm[1], tm[2], tm[3]);
  } else {
    const int64_t total = rows * dm;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (dtype == SA_BF16)
      gate_simt_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(
          rows, dm, (const __nv_bfloat16*)y_sa, (const __nv_bfloat16*)y_swa, ld_y,
          (const __nv_bfloat16*)w_sa, (const __nv_bfloat16*)w_swa, (__nv_bfloat16*)out, ld_out);
    else
      gate_simt_kernel<float><<<blocks, 256, 0, st>>>(rows, dm, (const float*)y_sa,
                                                      (const float*)y_swa, ld_y, (const float*)w_sa,
                                                      (const float*)w_swa, (float*)out, ld_out);
  }
  bump_launches();
  return cudaGetLastError() == cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
