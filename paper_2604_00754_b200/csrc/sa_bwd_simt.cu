// Backward pass on the CUDA cores (fp32 arithmetic, fp32 or bf16 storage), three kernels:
//   1. delta:   D_x[i] = g_x * sum_c dY[i,c] Y_x[i,c] per branch x, plus per-block partial
//               sums of dY.Y_x from which the gate-logit gradients are reduced in a fixed
//               order (no floating-point atomics anywhere: results are run-to-run identical);
//   2. dq:      one warp per query token walks its visible keys in both branches;
//   3. dk/dv:   one warp per key token walks the queries that see it, in both branches and
//               over the query heads of its GQA group.
// Formulas: derivative of Eq. 1 / Eq. 5 with the permutation held constant,
//   P_ij = exp(scale q_i.k_j - lse_i), dS_ij = P_ij (dY_x[i].V_j - D_x[i]).
#include <type_traits>

#include "sa_bwd_tc.cuh"
#include "sa_common.cuh"

namespace sa {
namespace {

constexpr int kWarps = 8;
constexpr int kMaxColsPerLane = 8;
constexpr int kDeltaRowsPerBlock = 64;

template <typename T>
__device__ __forceinline__ float dot_f32_row(const float* __restrict__ s, const T* __restrict__ row,
                                             int d) {
  float acc = 0.f;
  for (int c = 0; c < d; c += 4) {
    const float4 sv = *reinterpret_cast<const float4*>(s + c);
    acc = fmaf(sv.x, to_f32(row[c]), acc);
    acc = fmaf(sv.y, to_f32(row[c + 1]), acc);
    acc = fmaf(sv.z, to_f32(row[c + 2]), acc);
    acc = fmaf(sv.w, to_f32(row[c + 3]), acc);
  }
  return acc;
}

__device__ __forceinline__ float sigmoidf(float x) { return 1.f / (1.f + __expf(-x)); }

template <typename T>
__global__ void __launch_bounds__(kWarps * 32) bwd_delta_kernel(const BwdArgs a) {
  __shared__ float wsum[kWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hq = blockIdx.y, b = blockIdx.z % a.B, x = blockIdx.z / a.B;
  const float g = a.gate_logits ? sigmoidf(a.gate_logits[x * a.Hq + hq]) : 1.f;
  const T* dy = (const T*)a.dy + b * a.qs[0] + hq * a.qs[1];
  const T* yx = (const T*)a.y_x[x] + b * a.qs[0] + hq * a.qs[1];
  float* delta = a.delta + (((size_t)x * a.B + b) * a.Hq + hq) * a.n;
  float block_part = 0.f;
  for (int r = warp; r < kDeltaRowsPerBlock; r += kWarps) {
    const int i = blockIdx.x * kDeltaRowsPerBlock + r;
    if (i >= a.n) break;
    float dot = 0.f;
    for (int c = lane; c < a.d; c += 32)
      dot = fmaf(to_f32(dy[i * a.qs[2] + c]), to_f32(yx[i * a.qs[2] + c]), dot);
    dot = warp_sum(dot);
    if (lane == 0) delta[i] = g * dot;
    block_part += dot;
  }
  if (lane == 0) wsum[warp] = block_part;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int wv = 0; wv < kWarps; ++wv) s += wsum[wv];
    a.partials[(((size_t)x * a.B + b) * a.Hq + hq) * a.chunks + blockIdx.x] = s;
  }
}

__global__ void dgate_kernel(const BwdArgs a) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 2 * a.Hq) return;
  const int x = idx / a.Hq, hq = idx % a.Hq;
  float s = 0.f;
  for (int b = 0; b < a.B; ++b) {
    const float* p = a.partials + (((size_t)x * a.B + b) * a.Hq + hq) * a.chunks;
    for (int c = 0; c < a.chunks; ++c) s += p[c];
  }
  const float g = sigmoidf(a.gate_logits[idx]);
  a.dgate[idx] = g * (1.f - g) * s;
}

template <typename T>
__global__ void __launch_bounds__(kWarps * 32) bwd_dq_kernel(const BwdArgs a) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* qs = smem + warp * 2 * a.d;
  float* dys = qs + a.d;
  const int tok = blockIdx.x * kWarps + warp;
  const int hq = blockIdx.y, b = blockIdx.z;
  if (tok >= a.n) return;
  if (a.abort_flag && *a.abort_flag) return;
  const int hk = hq / (a.Hq / a.Hkv);
  const int64_t qoff = b * a.qs[0] + hq * a.qs[1] + tok * a.qs[2];
  const T* kbase = (const T*)a.k + b * a.ks[0] + hk * a.ks[1];
  const T* vbase = (const T*)a.v + b * a.ks[0] + hk * a.ks[1];
  const float scale2 = a.scale * kLog2e;
  for (int c = lane; c < a.d; c += 32) {
    qs[c] = to_f32(((const T*)a.q)[qoff + c]) * scale2;
    dys[c] = to_f32(((const T*)a.dy)[qoff + c]);
  }
  __syncwarp();

  float acc[kMaxColsPerLane];
#pragma unroll
  for (int x = 0; x < kMaxColsPerLane; ++x) acc[x] = 0.f;

  for (int x = 0; x < a.nbranch; ++x) {
    const bool swa = x == 1;
    const int32_t* perm = swa ? nullptr : a.perm + (size_t)b * a.n;
    const int slot = swa ? tok : a.inv[(size_t)b * a.n + tok];
    const MaskGeom g = make_geom(a.n, a.w, a.flags, swa);
    const SlotRange r = key_range(g, slot);
    const size_t row = (((size_t)x * a.B + b) * a.Hq + hq) * a.n + tok;
    const float lse2 = a.lse_x[x][((size_t)b * a.Hq + hq) * a.n + tok] * kLog2e;
    const float delta = a.delta[row];
    const float gx = a.gate_logits ? sigmoidf(a.gate_logits[x * a.Hq + hq]) : 1.f;
    for (int t0 = 0; t0 < r.count; t0 += 32) {
      const int t = t0 + lane;
      int ks = r.start + t, kt = -1;
      bool ok = t < r.count;
      if (ok) {
        if (r.wrap) ks = wrap_slot(ks, a.n);
        else ok = ks >= 0 && ks < a.n;
      }
      if (ok) {
        kt = perm ? perm[ks] : ks;
        ok = visible(g, slot, tok, ks, kt);
      }
      float ds = 0.f;
      if (ok) {
        const float p = exp2f(dot_f32_row<T>(qs, kbase + kt * a.ks[2], a.d) - lse2);
        const float dp = gx * dot_f32_row<T>(dys, vbase + kt * a.ks[2], a.d);
        ds = p * (dp - delta);
      }
      for (uint32_t rest = __ballot_sync(0xffffffffu, ok); rest; rest &= rest - 1) {
        const int src = __ffs(rest) - 1;
        const float dsj = __shfl_sync(0xffffffffu, ds, src);
        const int jt = __shfl_sync(0xffffffffu, kt, src);
        const T* kr = kbase + jt * a.ks[2];
#pragma unroll
        for (int y = 0; y < kMaxColsPerLane; ++y) {
          const int c = lane + 32 * y;
          if (c < a.d) acc[y] = fmaf(dsj, to_f32(kr[c]), acc[y]);
        }
      }
    }
  }
#pragma unroll
  for (int y = 0; y < kMaxColsPerLane; ++y) {
    const int c = lane + 32 * y;
    if (c < a.d) ((T*)a.dq)[qoff + c] = from_f32<T>(acc[y] * a.scale);
  }
}

template <typename T>
__global__ void __launch_bounds__(kWarps * 32) bwd_dkv_kernel(const BwdArgs a) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* ksm = smem + warp * 2 * a.d;
  float* vsm = ksm + a.d;
  const int tok = blockIdx.x * kWarps + warp;  // key token
  const int hk = blockIdx.y, b = blockIdx.z;
  if (tok >= a.n) return;
  if (a.abort_flag && *a.abort_flag) return;
  const int G = a.Hq / a.Hkv;
  const int64_t koff = b * a.ks[0] + hk * a.ks[1] + tok * a.ks[2];
  const float scale2 = a.scale * kLog2e;
  for (int c = lane; c < a.d; c += 32) {
    ksm[c] = to_f32(((const T*)a.k)[koff + c]) * scale2;
    vsm[c] = to_f32(((const T*)a.v)[koff + c]);
  }
  __syncwarp();

  float dk[kMaxColsPerLane], dv[kMaxColsPerLane];
#pragma unroll
  for (int y = 0; y < kMaxColsPerLane; ++y) dk[y] = dv[y] = 0.f;

  for (int x = 0; x < a.nbranch; ++x) {
    const bool swa = x == 1;
    const int32_t* perm = swa ? nullptr : a.perm + (size_t)b * a.n;
    const int kslot = swa ? tok : a.inv[(size_t)b * a.n + tok];
    const MaskGeom g = make_geom(a.n, a.w, a.flags, swa);
    const SlotRange r = query_range(g, kslot);
    for (int hq = hk * G; hq < (hk + 1) * G; ++hq) {
      const float gx = a.gate_logits ? sigmoidf(a.gate_logits[x * a.Hq + hq]) : 1.f;
      const T* qbase = (const T*)a.q + b * a.qs[0] + hq * a.qs[1];
      const T* dybase = (const T*)a.dy + b * a.qs[0] + hq * a.qs[1];
      const float* lse = a.lse_x[x] + ((size_t)b * a.Hq + hq) * a.n;
      const float* delta = a.delta + (((size_t)x * a.B + b) * a.Hq + hq) * a.n;
      for (int t0 = 0; t0 < r.count; t0 += 32) {
        const int t = t0 + lane;
        int qsl = r.start + t, qt = -1;
        bool ok = t < r.count;
        if (ok) {
          if (r.wrap) qsl = wrap_slot(qsl, a.n);
          else ok = qsl >= 0 && qsl < a.n;
        }
        if (ok) {
          qt = perm ? perm[qsl] : qsl;
          ok = visible(g, qsl, qt, kslot, tok);
        }
        float p = 0.f, ds = 0.f;
        if (ok) {
          p = exp2f(dot_f32_row<T>(ksm, qbase + qt * a.qs[2], a.d) - lse[qt] * kLog2e);
          const float dp = gx * dot_f32_row<T>(vsm, dybase + qt * a.qs[2], a.d);
          ds = p * (dp - delta[qt]);
          p *= gx;  // dV_j += P_ij * (g_x dY_i)
        }
        for (uint32_t rest = __ballot_sync(0xffffffffu, ok); rest; rest &= rest - 1) {
          const int src = __ffs(rest) - 1;
          const float pi = __shfl_sync(0xffffffffu, p, src);
          const float dsi = __shfl_sync(0xffffffffu, ds, src);
          const int it = __shfl_sync(0xffffffffu, qt, src);
          const T* qr = qbase + it * a.qs[2];
          const T* dyr = dybase + it * a.qs[2];
#pragma unroll
          for (int y = 0; y < kMaxColsPerLane; ++y) {
            const int c = lane + 32 * y;
            if (c < a.d) {
              dv[y] = fmaf(pi, to_f32(dyr[c]), dv[y]);
              dk[y] = fmaf(dsi, to_f32(qr[c]), dk[y]);
            }
          }
        }
      }
    }
  }
#pragma unroll
  for (int y = 0; y < kMaxColsPerLane; ++y) {
    const int c = lane + 32 * y;
    if (c < a.d) {
      ((T*)a.dk)[koff + c] = from_f32<T>(dk[y] * a.scale);
      ((T*)a.dv)[koff + c] = from_f32<T>(dv[y]);
    }
  }
}

inline size_t align_up(size_t x, size_t al) { return (x + al - 1) / al * al; }

template <typename T>
cudaError_t launch_all(const BwdArgs& a, cudaStream_t st) {
  const size_t smem = (size_t)kWarps * 2 * a.d * sizeof(float);
  bwd_delta_kernel<T><<<dim3(a.chunks, a.Hq, a.B * a.nbranch), kWarps * 32, 0, st>>>(a);
  bump_launches();
  if (a.gate_logits && a.dgate) {
    dgate_kernel<<<(2 * a.Hq + 127) / 128, 128, 0, st>>>(a);
    bump_launches();
  }
  if (tc_backward_supported(a, std::is_same<T, float>::value ? SA_F32 : SA_BF16))
    return launch_bwd_tc(a, st);      // dq, dk, dv on the tensor cores
  bwd_dq_kernel<T><<<dim3((a.n + kWarps - 1) / kWarps, a.Hq, a.B), kWarps * 32, smem, st>>>(a);
  bwd_dkv_kernel<T><<<dim3((a.n + kWarps - 1) / kWarps, a.Hkv, a.B), kWarps * 32, smem, st>>>(a);
  bump_launches(2);
  return cudaGetLastError();
}

}  // namespace

size_t bwd_ws_bytes(int B, int Hq, int n, int* chunks_out) {
  const int chunks = (n + kDeltaRowsPerBlock - 1) / kDeltaRowsPerBlock;
  if (chunks_out) *chunks_out = chunks;
  return align_up((size_t)2 * B * Hq * n * sizeof(float), 256) +
         align_up((size_t)2 * B * Hq * chunks * sizeof(float), 256);
}

cudaError_t launch_bwd_simt(const BwdArgs& a, int dtype, cudaStream_t st) {
  return dtype == SA_F32 ? launch_all<float>(a, st) : launch_all<__nv_bfloat16>(a, st);
}

}  // namespace sa
