// Internal declarations shared by the translation units of the library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sa.h"

namespace sa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Mask geometry in slot space.  h = ceil(w/2)-1 is the half width of the symmetric
// window (2*dist < w  <=>  dist <= h); the one-sided SWA window reaches w-1 back.
struct MaskGeom {
  int n, w, h;
  bool causal, linear, one_sided;  // one_sided only ever set for the SWA branch
};

__host__ __device__ inline MaskGeom make_geom(int n, int w, uint32_t flags, bool swa) {
  MaskGeom g;
  g.n = n;
  g.w = w;
  g.h = (int)(((int64_t)w + 1) / 2 - 1);
  g.causal = flags & SA_CAUSAL;
  g.linear = flags & SA_LINEAR_WINDOW;
  g.one_sided = swa && (flags & SA_SWA_ONE_SIDED);
  return g;
}

// May the query (slot sq, token iq) see the key (slot sk, token jk)?  Exact integers.
__device__ __forceinline__ bool visible(const MaskGeom& g, int sq, int iq, int sk, int jk) {
  if (g.one_sided) {
    const int back = iq - jk;
    return back >= 0 && back <= g.w - 1;
  }
  int dist = sq > sk ? sq - sk : sk - sq;
  if (!g.linear) dist = min(dist, g.n - dist);
  if (2ll * dist >= (long long)g.w) return false;
  return !g.causal || jk <= iq;
}

// Slots a query at slot s has to look at: `count` slots starting at `start` (which may be
// negative or run past n-1; callers wrap modulo n when `wrap`, otherwise skip slots
// outside [0, n)).  Never visits a slot twice.
struct SlotRange {
  int start, count;
  bool wrap;
};

__host__ __device__ inline SlotRange key_range(const MaskGeom& g, int s) {
  SlotRange r;
  if (g.one_sided) {
    r.wrap = false;
    r.start = s - min(g.w - 1, g.n);
    r.count = s - r.start + 1;
  } else if (2ll * g.h + 1 >= g.n) {
    r.wrap = false;
    r.start = 0;
    r.count = g.n;
  } else {
    r.wrap = !g.linear;
    r.start = s - g.h;
    r.count = 2 * g.h + 1;
  }
  return r;
}

// Queries that can see a key at slot s (the transpose of key_range).
__host__ __device__ inline SlotRange query_range(const MaskGeom& g, int s) {
  SlotRange r;
  if (g.one_sided) {
    r.wrap = false;
    r.start = s;
    r.count = min(g.w - 1, g.n) + 1;
  } else {
    r = key_range(g, s);
  }
  return r;
}

__device__ __forceinline__ int wrap_slot(int slot, int n) {
  slot %= n;
  return slot < 0 ? slot + n : slot;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Device address of the status word of the current device (lives in the library image);
// null if the runtime call that resolves it failed.
int* status_ptr();
void bump_launches(uint64_t k = 1);
// Current value of a test hook (sa_debug_key); see sa_debug_set.
int debug_option(int key);

struct FwdArgs {
  const void *q, *k, *v;
  const int32_t *perm, *inv;  // null for the SWA branch
  void* y;                    // final output rows
  void* y_branch;             // nullable: this branch's own (ungated) output
  float* lse;                 // nullable
  const void* y_other;        // nullable: the other branch's finished output (gated combine)
  const float *rope_cos, *rope_sin;  // nullable [n, d/2]: rotate Q and K rows inside the gather
  const float* gate_logits;   // nullable [2,Hq]
  int B, Hq, Hkv, n, d, w;
  uint32_t flags;
  float scale;
  int64_t qs[3], ks[3];
  bool swa;
  const int* abort_flag;  // nullable: kernels return at once when it reads non-zero
};

struct BwdArgs {
  const void *q, *k, *v, *dy;
  const int32_t *perm, *inv;
  const float* gate_logits;  // nullable
  const void* y_x[2];        // branch outputs (0 = SA, 1 = SWA)
  const float* lse_x[2];
  void *dq, *dk, *dv;
  float* dgate;
  float* delta;     // ws: [2,B,Hq,n]
  float* partials;  // ws: [2,B,Hq,chunks]
  int chunks;
  int B, Hq, Hkv, n, d, w;
  uint32_t flags;
  float scale;
  int64_t qs[3], ks[3];
  int nbranch;
  const int* abort_flag;  // nullable: kernels return at once when it reads non-zero
};

// Launchers (each returns cudaGetLastError() of its launches).
cudaError_t launch_make_perm(uint64_t seed, uint32_t layer, int B, int n, int32_t* perm,
                             int32_t* inv, void* ws, cudaStream_t st);
size_t make_perm_ws_bytes(int B, int n);

cudaError_t launch_fwd_simt(const FwdArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_validate_perm(const int32_t* perm, const int32_t* inv, int B, int n,
                                 cudaStream_t st);

cudaError_t launch_rope_apply(const void* x, void* out, int B, int H, int n, int d,
                              const int64_t s[3], int dtype, const float* cs, const float* sn,
                              bool inverse, cudaStream_t st);

bool gate_forward_wide(int64_t rows, int dm, const void* y_sa, const void* y_swa, int64_t ld_y,
                       const void* w_sa, const void* w_swa, void* out, int64_t ld_out,
                       int* status, int sms, cudaStream_t st, cudaError_t* err);

cudaError_t launch_bwd_simt(const BwdArgs& a, int dtype, cudaStream_t st);
size_t bwd_ws_bytes(int B, int Hq, int n, int* chunks_out);

cudaError_t launch_coverage(int L, int n, int w, uint32_t flags, const int32_t* perm,
                            const int32_t* inv, int src, int64_t* nnz, int32_t* row_count,
                            int32_t* reach, void* ws, cudaStream_t st);
size_t coverage_ws_bytes(int L, int n);

}  // namespace sa
