// Backward of the projection gates (Eq. 5-6): with z = y w^T, g = sigmoid(z), out = g * y,
//   dz = dout * y * g * (1 - g),   dw = dz^T y,   dy = dout * g + dz w      (per path).
// Three contractions per path, all on the 5th-generation tensor cores through one kernel
// template (128 x 256 output tiles, or 128 x 128 for small products, TMA ring,
// double-buffered fp32 accumulators in tensor memory, eight epilogue warps):
//   kDz: z = y w^T        (both operands K-major);  epilogue writes dz and dout * g
//   kDy: dz w             (w read with its rows as the contraction index: N-major operand);
//                          epilogue adds dout * g and writes dy
//   kDw: dz^T y           (both operands read with their rows as the contraction index);
//                          epilogue writes dw
// A plain kernel per step serves fp32 and sizes the tensor-core path does not take.
//
// Every mbarrier wait is bounded; on expiry the CTA records SA_ERR_TIMEOUT in the device
// status word, stops issuing work, drains what it started and returns.
#include "sa_gemm_common.cuh"

namespace sa {
namespace {

enum BwdMode { kDz = 0, kDy = 1, kDw = 2, kFwd = 3 };   // kFwd: the forward's sigmoid(y w^T) * y

constexpr int kT = 128, kBK = 64;                  // output tiles of 128 rows, K chunks of 64
constexpr int kATileBytes = kT * kBK * 2;          // A of one K chunk, either major: 16 KB
constexpr int kChunk = 64 * kBK * 2;               // 64 rows x 64 columns: one box of a row-contracted operand
constexpr int kRingBytes = 12 * kATileBytes;       // 192 KB of operand stages
// TN: columns of the output tile.  256 halves the operand bytes per flop of the B side and is
// used when it still leaves at least one tile per SM; 128 otherwise.  A stage holds 64 KB or
// 48 KB (two K chunks of A + B at TN = 128, one at TN = 256): eight or four products.
template <int TN> struct Tile {
  static constexpr int kCps = TN == 128 ? 2 : 1;                 // K chunks per stage
  static constexpr int kBTileBytes = TN * kBK * 2;
  static constexpr int kStageBytes = kCps * (kATileBytes + kBTileBytes);
  static constexpr int kStages = kRingBytes / kStageBytes;       // 3 or 4
};
constexpr int kMaxStages = 4;
constexpr int kThreadsB = 320;
constexpr int kOffBars = kRingBytes;
constexpr int kBarFull = 0, kBarEmpty = kMaxStages, kBarAccFull = 2 * kMaxStages,
              kBarAccEmpty = 2 * kMaxStages + 2, kNumBars = 2 * kMaxStages + 4;
constexpr int kOffMisc = kOffBars + kNumBars * 8;
constexpr int kSmemB = kOffMisc + 16;

struct BwdGateParams {
  // epilogue operands, all [*, dm] with the given pitches (elements)
  const __nv_bfloat16 *dout, *y;   // kDz
  __nv_bfloat16 *dz, *dyd;         // kDz out; kDy reads dyd
  __nv_bfloat16* out;              // kDy: dy, kDw: dw
  int64_t ld_y, ld_ws, ld_out;
  int64_t m_rows, n_cols;          // extent of the product
  int tiles_m, tiles_n, k_pairs;   // k_pairs: hand-overs per tile (one or two K chunks each)
  int accum;                       // kFwd: add to what out already holds (second path)
  int* status;
};

__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc,
                                       uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc)
      : "memory");
}
// bit 15: A is MN-major, bit 16: B is MN-major
__host__ __device__ constexpr uint32_t idesc_of(int tn, bool a_mn, bool b_mn) {
  return instr_desc(kT, tn, b_mn) | ((a_mn ? 1u : 0u) << 15);
}
template <int MODE, int TN>
__global__ void __launch_bounds__(kThreadsB, 1)
gate_bwd_kernel(const __grid_constant__ BwdGateParams p, const __grid_constant__ CUtensorMap tm_a,
                const __grid_constant__ CUtensorMap tm_b) {
  constexpr bool kAmn = MODE == kDw, kBmn = MODE == kDy || MODE == kDw;
  using TL = Tile<TN>;
  constexpr int kStages = TL::kStages, kStageBytes = TL::kStageBytes, kTN = TN;
  constexpr int kBlock = 2048 / TN;       // column tiles per block of the tile order
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {
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
    for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), (i >= kBarAccEmpty) ? 256 : 1);
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
  // blocks of 2048 columns, row tile by row tile inside a block (operand slices stay in L2)
  auto origin = [&](int tile, int* m0, int* n0) {
    const int per_block = p.tiles_m * kBlock;
    const int nb = tile / per_block, rem = tile - nb * per_block;
    const int width = min(kBlock, p.tiles_n - nb * kBlock);
    *m0 = (rem / width) * kT;
    *n0 = (nb * kBlock + rem % width) * kTN;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t use = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        int m0, n0;
        origin(tile, &m0, &n0);
        for (int kp = 0; kp < p.k_pairs && ok; ++kp, ++use) {
          const uint32_t s = use % kStages;
          if (use >= (uint32_t)kStages)
            ok = mbar_wait(bar(kBarEmpty + s), (use / kStages - 1) & 1u, gave_up, p.status);
          if (!ok) break;
          const uint32_t dst = sbase + s * kStageBytes, fb = bar(kBarFull + s);
          mbar_expect_tx(fb, kStageBytes);
#pragma unroll
          for (int q = 0; q < TL::kCps; ++q) {
            const int k0 = (TL::kCps * kp + q) * kBK;                   // past the end: zeros
            const uint32_t da = dst + q * (kATileBytes + TL::kBTileBytes), db = da + kATileBytes;
            if (kAmn) {
#pragma unroll
              for (int c = 0; c < kT / 64; ++c) tma_load_2d(da + c * kChunk, &tm_a, m0 + 64 * c, k0, fb);
            } else {
              tma_load_2d(da, &tm_a, k0, m0, fb);
            }
            if (kBmn) {
#pragma unroll
              for (int c = 0; c < kTN / 64; ++c) tma_load_2d(db + c * kChunk, &tm_b, n0 + 64 * c, k0, fb);
            } else {
              tma_load_2d(db, &tm_b, k0, n0, fb);
            }
          }
        }
      }
      if (!ok || *gave_up) {   // loads started but never consumed must land before smem goes
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
      constexpr uint32_t idesc = idesc_of(TN, kAmn, kBmn);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t kLoK = (16u >> 4) << 16;                       // K-major operand
      constexpr uint32_t kLoMN = ((uint32_t)kChunk >> 4) << 16;           // next 64 columns
      constexpr uint32_t kStepK = 32u >> 4, kStepMN = 2048u >> 4;         // one K step of 16
      uint32_t use = 0, it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++it) {
        const uint32_t buf = it & 1u;
        if (it >= 2)
          ok = mbar_wait(bar(kBarAccEmpty + buf), (it / 2 - 1) & 1u, gave_up, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d = tmem + buf * kTN;
        for (int kp = 0; kp < p.k_pairs && ok; ++kp, ++use) {
          const uint32_t s = use % kStages;
          ok = mbar_wait(bar(kBarFull + s), (use / kStages) & 1u, gave_up, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t lo = (sbase + s * kStageBytes) >> 4;
#pragma unroll
          for (int q = 0; q < TL::kCps; ++q) {
            const uint32_t la = lo + q * ((kATileBytes + TL::kBTileBytes) >> 4);
            const uint64_t a0 = desc64(la | (kAmn ? kLoMN : kLoK), kDescHi);
            const uint64_t b0 = desc64((la + (kATileBytes >> 4)) | (kBmn ? kLoMN : kLoK), kDescHi);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_ss(d, a0 + ks * (kAmn ? kStepMN : kStepK), b0 + ks * (kBmn ? kStepMN : kStepK),
                     idesc, (kp > 0 || q > 0 || ks > 0) ? 1u : 0u);
          }
          tc_commit(bar(kBarEmpty + s));
        }
        if (ok) tc_commit(bar(kBarAccFull + buf));
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------- epilogue (warps 2-9)
    const int half = (warp - 2) >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
      const uint32_t buf = it & 1u;
      int m0, n0;
      origin(tile, &m0, &n0);
      ok = mbar_wait(bar(kBarAccFull + buf), (it / 2) & 1u, gave_up, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int64_t r = (int64_t)m0 + row;
      const bool row_ok = r < p.m_rows;
#pragma unroll 1
      for (int c = (kTN / 64) * half; c < (kTN / 64) * (half + 1); ++c) {
        uint32_t acc[32];
        tmem_ld32(tmem + lane_addr + buf * kTN + 32 * c, acc);
        tmem_wait_ld();
        const int col = n0 + 32 * c;
        // the epilogue's row reads are requested together, ahead of the stores they may not
        // pass (the outputs may alias the inputs as far as the compiler knows), so that their
        // latencies overlap: fy = y (kDz, kFwd) or dout * g (kDy), fo = dout (kDz) or out (kFwd)
        uint4 fy[4], fo[4];
        if (MODE != kDw && row_ok && col < p.n_cols) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            const int64_t e = col + 8 * x8;
            if (MODE == kDy) fy[x8] = *reinterpret_cast<const uint4*>(p.dyd + r * p.ld_ws + e);
            else fy[x8] = *reinterpret_cast<const uint4*>(p.y + r * p.ld_y + e);
            if (MODE == kDz || (MODE == kFwd && p.accum))
              fo[x8] = *reinterpret_cast<const uint4*>((MODE == kDz ? p.dout : p.out) + r * p.ld_out + e);
          }
        }
        if (row_ok && col < p.n_cols) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            const int64_t e = col + 8 * x8;
            float v8[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) v8[x] = __uint_as_float(acc[8 * x8 + x]);
            uint4 st;
            __nv_bfloat162* hs = reinterpret_cast<__nv_bfloat162*>(&st);
            if (MODE == kDz) {
              const __nv_bfloat162* hy = reinterpret_cast<const __nv_bfloat162*>(&fy[x8]);
              const __nv_bfloat162* hd = reinterpret_cast<const __nv_bfloat162*>(&fo[x8]);
              uint4 st2;
              __nv_bfloat162* hs2 = reinterpret_cast<__nv_bfloat162*>(&st2);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                const float g0 = logistic(v8[2 * x]), g1 = logistic(v8[2 * x + 1]);
                const float d0 = __low2float(hd[x]), d1 = __high2float(hd[x]);
                hs[x] = __floats2bfloat162_rn(d0 * __low2float(hy[x]) * g0 * (1.f - g0),
                                              d1 * __high2float(hy[x]) * g1 * (1.f - g1));
                hs2[x] = __floats2bfloat162_rn(d0 * g0, d1 * g1);
              }
              *reinterpret_cast<uint4*>(p.dz + r * p.ld_ws + e) = st;
              *reinterpret_cast<uint4*>(p.dyd + r * p.ld_ws + e) = st2;
            } else if (MODE == kFwd) {
              const __nv_bfloat162* hy = reinterpret_cast<const __nv_bfloat162*>(&fy[x8]);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                v8[2 * x] = logistic(v8[2 * x]) * __low2float(hy[x]);
                v8[2 * x + 1] = logistic(v8[2 * x + 1]) * __high2float(hy[x]);
              }
              uint4* dst = reinterpret_cast<uint4*>(p.out + r * p.ld_out + e);
              if (p.accum) {
                const __nv_bfloat162* ho = reinterpret_cast<const __nv_bfloat162*>(&fo[x8]);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  v8[2 * x] += __low2float(ho[x]);
                  v8[2 * x + 1] += __high2float(ho[x]);
                }
              }
#pragma unroll
              for (int x = 0; x < 4; ++x) hs[x] = __floats2bfloat162_rn(v8[2 * x], v8[2 * x + 1]);
              *dst = st;
            } else {
              if (MODE == kDy) {
                const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&fy[x8]);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  v8[2 * x] += __low2float(hp[x]);
                  v8[2 * x + 1] += __high2float(hp[x]);
                }
              }
#pragma unroll
              for (int x = 0; x < 4; ++x) hs[x] = __floats2bfloat162_rn(v8[2 * x], v8[2 * x + 1]);
              *reinterpret_cast<uint4*>(p.out + r * p.ld_out + e) = st;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(kBarAccEmpty + buf));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u)
                 : "memory");
  }
}

// ------------------------------------------------- plain kernels (fp32, other sizes)

template <typename T>
__global__ void dz_simt_kernel(int64_t rows, int dm, const T* __restrict__ dout, int64_t ld_dout,
                               const T* __restrict__ y, int64_t ld_y, const T* __restrict__ w,
                               float* __restrict__ dz, float* __restrict__ dyd) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * dm) return;
  const int64_t r = idx / dm;
  const int o = (int)(idx % dm);
  const T* yr = y + r * ld_y;
  const T* wo = w + (int64_t)o * dm;
  float z = 0.f;
  for (int i = 0; i < dm; ++i) z = fmaf(to_f32(yr[i]), to_f32(wo[i]), z);
  const float g = 1.f / (1.f + expf(-z)), d = to_f32(dout[r * ld_dout + o]);
  dz[idx] = d * to_f32(yr[o]) * g * (1.f - g);
  dyd[idx] = d * g;
}

template <typename T>
__global__ void dy_simt_kernel(int64_t rows, int dm, const float* __restrict__ dz,
                               const float* __restrict__ dyd, const T* __restrict__ w,
                               T* __restrict__ dy, int64_t ld_dy) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * dm) return;
  const int64_t r = idx / dm;
  const int i = (int)(idx % dm);
  float acc = dyd[idx];
  for (int o = 0; o < dm; ++o) acc = fmaf(dz[r * dm + o], to_f32(w[(int64_t)o * dm + i]), acc);
  dy[r * ld_dy + i] = from_f32<T>(acc);
}

template <typename T>
__global__ void dw_simt_kernel(int64_t rows, int dm, const float* __restrict__ dz,
                               const T* __restrict__ y, int64_t ld_y, T* __restrict__ dw) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)dm * dm) return;
  const int o = (int)(idx / dm), i = (int)(idx % dm);
  float acc = 0.f;
  for (int64_t r = 0; r < rows; ++r) acc = fmaf(dz[r * dm + o], to_f32(y[r * ld_y + i]), acc);
  dw[idx] = from_f32<T>(acc);
}

// ------------------------------------------------------------------------------ host

// Wide (128 x 256) tiles when they still give every SM at least two tiles.
bool wide_tiles(int64_t m_rows, int64_t n_cols, int sms) {
  return ((m_rows + kT - 1) / kT) * ((n_cols + 255) / 256) >= 2 * (int64_t)sms;
}

template <int MODE, int TN>
cudaError_t launch_mode(BwdGateParams p, const CUtensorMap& a, const CUtensorMap& b, int64_t k,
                        int sms, cudaStream_t st) {
  p.tiles_m = (int)((p.m_rows + kT - 1) / kT);
  p.tiles_n = (int)((p.n_cols + TN - 1) / TN);
  const int per = Tile<TN>::kCps * kBK;
  p.k_pairs = (int)((k + per - 1) / per);
  cudaError_t e = cudaFuncSetAttribute(gate_bwd_kernel<MODE, TN>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemB);
  if (e != cudaSuccess) return e;
  const int64_t total = (int64_t)p.tiles_m * p.tiles_n;
  const unsigned grid = (unsigned)(total < sms ? total : sms);
  gate_bwd_kernel<MODE, TN><<<grid, kThreadsB, kSmemB, st>>>(p, a, b);
  bump_launches();
  return cudaGetLastError();
}

}  // namespace

// Forward of one or two paths with 128 x 256 tiles, one launch per path (the second adds to
// the first's rounded result); false when the product is too small for wide tiles to fill
// the GPU, and the caller's fused kernel should run instead.
bool gate_forward_wide(int64_t rows, int dm, const void* y_sa, const void* y_swa, int64_t ld_y,
                       const void* w_sa, const void* w_swa, void* out, int64_t ld_out,
                       int* status, int sms, cudaStream_t st, cudaError_t* err) {
  *err = cudaSuccess;
  if (!wide_tiles(rows, dm, sms)) return false;
  for (int x = 0; x < (y_swa ? 2 : 1); ++x) {
    const void* y = x ? y_swa : y_sa;
    const void* w = x ? w_swa : w_sa;
    CUtensorMap y_k, w_k;
    if (!make_map(&y_k, y, rows, dm, ld_y, 128) || !make_map(&w_k, w, dm, dm, dm, 256)) {
      *err = cudaErrorUnknown;
      return true;
    }
    BwdGateParams p{};
    p.status = status;
    p.y = (const __nv_bfloat16*)y; p.ld_y = ld_y;
    p.out = (__nv_bfloat16*)out; p.ld_out = ld_out;
    p.m_rows = rows; p.n_cols = dm;
    p.accum = x;
    *err = launch_mode<kFwd, 256>(p, y_k, w_k, dm, sms, st);
    if (*err != cudaSuccess) return true;
  }
  return true;
}

}  // namespace sa

extern "C" size_t sa_gate_projection_backward_ws_bytes(int64_t rows, int32_t dm) {
  if (rows < 1 || dm < 1) return (size_t)-1;
  return (size_t)rows * (size_t)dm * 2u * sizeof(float);    // dz and dout * g, fp32 at most
}

extern "C" sa_status sa_gate_projection_backward(
    int64_t rows, int32_t dm, int32_t dtype, const void* dout, int64_t ld_dout, const void* y_sa,
    const void* y_swa, int64_t ld_y, const void* w_sa, const void* w_swa, void* dy_sa,
    void* dy_swa, int64_t ld_dy, void* dw_sa, void* dw_swa, void* ws, size_t ws_bytes,
    sa_stream_t stream) {
  using namespace sa;
  if (rows < 1 || dm < 1 || ld_y < dm || ld_dout < dm || ld_dy < dm) return SA_ERR_INVALID_ARG;
  if (!dout || !y_sa || !w_sa || !dy_sa || !dw_sa || !ws) return SA_ERR_INVALID_ARG;
  if (y_swa && (!w_swa || !dy_swa || !dw_swa)) return SA_ERR_INVALID_ARG;
  if (dtype != SA_F32 && dtype != SA_BF16) return SA_ERR_INVALID_ARG;
  if (ws_bytes < sa_gate_projection_backward_ws_bytes(rows, dm)) return SA_ERR_WORKSPACE;
  if (rows * (int64_t)dm > (1ll << 40)) return SA_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc_off = debug_option(SA_DEBUG_TENSOR_CORES) == 0;
  bool tc = !tc_off && dtype == SA_BF16 && dm % 64 == 0 && ld_y % 8 == 0 && ld_dout % 8 == 0 &&
            ld_dy % 8 == 0 && rows < (1ll << 31) - 256 && aligned16(ws) && aligned16(dout);
  const void* ptrs[] = {y_sa, w_sa, dy_sa, dw_sa, y_swa, w_swa, dy_swa, dw_swa};
  for (const void* q : ptrs) tc = tc && aligned16(q);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SA_ERR_CUDA;
  int* status = status_ptr();
  if (!status) return SA_ERR_CUDA;

  for (int x = 0; x < (y_swa ? 2 : 1); ++x) {
    const void* y = x ? y_swa : y_sa;
    const void* w = x ? w_swa : w_sa;
    void* dy = x ? dy_swa : dy_sa;
    void* dw = x ? dw_swa : dw_sa;
    if (tc) {
      __nv_bfloat16* dz = (__nv_bfloat16*)ws;
      __nv_bfloat16* dyd = dz + rows * (int64_t)dm;
      const bool wide_r = wide_tiles(rows, dm, sms), wide_w = wide_tiles(dm, dm, sms);
      CUtensorMap y_k, w_k, dz_k, w_mn, dz_mn, y_mn;
      if (!make_map(&y_k, y, rows, dm, ld_y, 128) ||
          !make_map(&w_k, w, dm, dm, dm, wide_r ? 256 : 128) ||
          !make_map(&dz_k, dz, rows, dm, dm, 128) || !make_map(&w_mn, w, dm, dm, dm, 64) ||
          !make_map(&dz_mn, dz, rows, dm, dm, 64) || !make_map(&y_mn, y, rows, dm, ld_y, 64))
        return SA_ERR_CUDA;
      BwdGateParams p{};
      p.status = status;
      p.dz = dz; p.dyd = dyd; p.ld_ws = dm; p.ld_y = ld_y;
      // z = y w^T; epilogue: dz, dout * g
      p.dout = (const __nv_bfloat16*)dout; p.y = (const __nv_bfloat16*)y; p.ld_out = ld_dout;
      p.m_rows = rows; p.n_cols = dm;
      if ((wide_r ? launch_mode<kDz, 256>(p, y_k, w_k, dm, sms, st)
                  : launch_mode<kDz, 128>(p, y_k, w_k, dm, sms, st)) != cudaSuccess)
        return SA_ERR_CUDA;
      // dy = dz w + dout * g
      p.out = (__nv_bfloat16*)dy; p.ld_out = ld_dy;
      if ((wide_r ? launch_mode<kDy, 256>(p, dz_k, w_mn, dm, sms, st)
                  : launch_mode<kDy, 128>(p, dz_k, w_mn, dm, sms, st)) != cudaSuccess)
        return SA_ERR_CUDA;
      // dw = dz^T y
      p.out = (__nv_bfloat16*)dw; p.ld_out = dm;
      p.m_rows = dm; p.n_cols = dm;
      if ((wide_w ? launch_mode<kDw, 256>(p, dz_mn, y_mn, rows, sms, st)
                  : launch_mode<kDw, 128>(p, dz_mn, y_mn, rows, sms, st)) != cudaSuccess)
        return SA_ERR_CUDA;
    } else {
      float* dz = (float*)ws;
      float* dyd = dz + rows * (int64_t)dm;
      const unsigned b1 = (unsigned)((rows * dm + 255) / 256);
      const unsigned b2 = (unsigned)(((int64_t)dm * dm + 255) / 256);
      if (dtype == SA_BF16) {
        typedef __nv_bfloat16 T;
        dz_simt_kernel<T><<<b1, 256, 0, st>>>(rows, dm, (const T*)dout, ld_dout, (const T*)y, ld_y,
                                              (const T*)w, dz, dyd);
        dy_simt_kernel<T><<<b1, 256, 0, st>>>(rows, dm, dz, dyd, (const T*)w, (T*)dy, ld_dy);
        dw_simt_kernel<T><<<b2, 256, 0, st>>>(rows, dm, dz, (const T*)y, ld_y, (T*)dw);
      } else {
        typedef float T;
        dz_simt_kernel<T><<<b1, 256, 0, st>>>(rows, dm, (const T*)dout, ld_dout, (const T*)y, ld_y,
                                              (const T*)w, dz, dyd);
        dy_simt_kernel<T><<<b1, 256, 0, st>>>(rows, dm, dz, dyd, (const T*)w, (T*)dy, ld_dy);
        dw_simt_kernel<T><<<b2, 256, 0, st>>>(rows, dm, dz, (const T*)y, ld_y, (T*)dw);
      }
      bump_launches(3);
      if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    }
  }
  return SA_OK;
}
