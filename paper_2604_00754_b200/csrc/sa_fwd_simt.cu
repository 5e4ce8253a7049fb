// General forward kernel on the CUDA cores: any d (multiple of 8, <= 256), fp32 or bf16
// storage, fp32 arithmetic.  It serves the fp32 configuration (a single-pass TF32 product
// cannot hold 1e-4 max-abs error), odd shapes and strides, and is the on-device cross-check
// of the tensor-core path.
//
// One warp owns one query row (Eq. 1 for one i).  Keys are taken 32 at a time in slot
// order: each lane scores one key (gathered through perm for the SA branch), the warp
// keeps an online softmax, then the 32 weighted value rows are accumulated with each lane
// owning output columns lane, lane+32, ...  The finished row is scattered to its original
// position, optionally combined with the other branch through the gate of Eq. 5.
#include "sa_common.cuh"

namespace sa {
namespace {

constexpr int kWarps = 8;
constexpr int kMaxColsPerLane = 8;  // d <= 256

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ qs, const T* __restrict__ row,
                                         int d);

template <>
__device__ __forceinline__ float dot_row<float>(const float* __restrict__ qs,
                                                const float* __restrict__ row, int d) {
  float acc = 0.f;
  for (int c = 0; c < d; c += 4) {
    const float4 kv = *reinterpret_cast<const float4*>(row + c);
    const float4 qv = *reinterpret_cast<const float4*>(qs + c);
    acc = fmaf(qv.x, kv.x, acc); acc = fmaf(qv.y, kv.y, acc);
    acc = fmaf(qv.z, kv.z, acc); acc = fmaf(qv.w, kv.w, acc);
  }
  return acc;
}

template <>
__device__ __forceinline__ float dot_row<__nv_bfloat16>(const float* __restrict__ qs,
                                                        const __nv_bfloat16* __restrict__ row,
                                                        int d) {
  float acc = 0.f;
  for (int c = 0; c < d; c += 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(row + c);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const float4 q0 = *reinterpret_cast<const float4*>(qs + c);
    const float4 q1 = *reinterpret_cast<const float4*>(qs + c + 4);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    const float2 e = __bfloat1622float2(h[2]), f = __bfloat1622float2(h[3]);
    acc = fmaf(q0.x, a.x, acc); acc = fmaf(q0.y, a.y, acc);
    acc = fmaf(q0.z, b.x, acc); acc = fmaf(q0.w, b.y, acc);
    acc = fmaf(q1.x, e.x, acc); acc = fmaf(q1.y, e.y, acc);
    acc = fmaf(q1.z, f.x, acc); acc = fmaf(q1.w, f.y, acc);
  }
  return acc;
}

template <typename T>
__global__ void __launch_bounds__(kWarps * 32) fwd_simt_kernel(const FwdArgs a) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* qs = smem + warp * a.d;

  const int slot = blockIdx.x * kWarps + warp;  // position in the order attention runs in
  const int hq = blockIdx.y, b = blockIdx.z;
  if (slot >= a.n) return;
  if (a.abort_flag && *a.abort_flag) return;  // an earlier check rejected perm/inv
  const int hk = hq / (a.Hq / a.Hkv);
  const int32_t* perm = a.swa ? nullptr : a.perm + (size_t)b * a.n;
  const int tok = perm ? perm[slot] : slot;

  const T* q = (const T*)a.q + b * a.qs[0] + hq * a.qs[1] + tok * a.qs[2];
  const T* kbase = (const T*)a.k + b * a.ks[0] + hk * a.ks[1];
  const T* vbase = (const T*)a.v + b * a.ks[0] + hk * a.ks[1];
  const float scale2 = a.scale * kLog2e;
  for (int c = lane; c < a.d; c += 32) qs[c] = to_f32(q[c]) * scale2;
  __syncwarp();

  const MaskGeom g = make_geom(a.n, a.w, a.flags, a.swa);
  const SlotRange r = key_range(g, slot);

  float acc[kMaxColsPerLane];
#pragma unroll
  for (int x = 0; x < kMaxColsPerLane; ++x) acc[x] = 0.f;
  float m = -INFINITY, l = 0.f;

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
    float s = -INFINITY;
    if (ok) s = dot_row<T>(qs, kbase + kt * a.ks[2], a.d);
    if (!__any_sync(0xffffffffu, ok)) continue;
    const float m_new = fmaxf(m, warp_max(s));       // finite: some lane is visible
    const float corr = exp2f(m - m_new);              // m = -inf gives 0
    const float p = ok ? exp2f(s - m_new) : 0.f;
    l = l * corr + warp_sum(p);
    m = m_new;
#pragma unroll
    for (int x = 0; x < kMaxColsPerLane; ++x) acc[x] *= corr;
    const uint32_t live = __ballot_sync(0xffffffffu, ok);
    for (uint32_t rest = live; rest; rest &= rest - 1) {
      const int src = __ffs(rest) - 1;
      const float pj = __shfl_sync(0xffffffffu, p, src);
      const int jt = __shfl_sync(0xffffffffu, kt, src);
      const T* vr = vbase + jt * a.ks[2];
#pragma unroll
      for (int x = 0; x < kMaxColsPerLane; ++x) {
        const int c = lane + 32 * x;
        if (c < a.d) acc[x] = fmaf(pj, to_f32(vr[c]), acc[x]);
      }
    }
  }

  const float inv_l = 1.f / l;
  float g_this = 1.f, g_other = 0.f;
  if (a.gate_logits) {
    const float l_sa = a.gate_logits[hq], l_swa = a.gate_logits[a.Hq + hq];
    const float s_sa = 1.f / (1.f + __expf(-l_sa)), s_swa = 1.f / (1.f + __expf(-l_swa));
    g_this = a.swa ? s_swa : s_sa;
    g_other = a.swa ? s_sa : s_swa;
  }
  const int64_t off = b * a.qs[0] + hq * a.qs[1] + tok * a.qs[2];
#pragma unroll
  for (int x = 0; x < kMaxColsPerLane; ++x) {
    const int c = lane + 32 * x;
    if (c < a.d) {
      float o = acc[x] * inv_l;
      if (a.y_branch) {
        const T ob = from_f32<T>(o);
        ((T*)a.y_branch)[off + c] = ob;
        o = to_f32(ob);  // combine what was stored, as the backward pass will read it
      }
      if (a.gate_logits) {
        o *= g_this;
        if (a.y_other) o = fmaf(g_other, to_f32(((const T*)a.y_other)[off + c]), o);
      }
      if (a.y) ((T*)a.y)[off + c] = from_f32<T>(o);
    }
  }
  if (a.lse && lane == 0)
    a.lse[((size_t)b * a.Hq + hq) * a.n + tok] = (m + log2f(l)) * kLn2;
}

}  // namespace

cudaError_t launch_fwd_simt(const FwdArgs& a, int dtype, cudaStream_t st) {
  const dim3 grid((a.n + kWarps - 1) / kWarps, a.Hq, a.B);
  const size_t smem = (size_t)kWarps * a.d * sizeof(float);
  if (dtype == SA_F32) fwd_simt_kernel<float><<<grid, kWarps * 32, smem, st>>>(a);
  else fwd_simt_kernel<__nv_bfloat16><<<grid, kWarps * 32, smem, st>>>(a);
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa
