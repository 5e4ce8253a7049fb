// Mask statistics and receptive-field growth (Sec. 3.2 and Prop. 2): per-query visible-key
// counts, their total, and the size of the set reachable from one token through L layers
// that each draw their own permutation.  Integer work only.
#include "sa_common.cuh"

namespace sa {
namespace {

// One warp per query token of one layer: counts the visible keys of its window and, when
// the token is in the current frontier, marks them in the next frontier.
__global__ void __launch_bounds__(256)
layer_kernel(int n, int w, uint32_t flags, const int32_t* __restrict__ perm,
             const int32_t* __restrict__ inv, const int32_t* __restrict__ cur,
             int32_t* __restrict__ nxt, int32_t* __restrict__ row_count,
             unsigned long long* __restrict__ nnz) {
  __shared__ int32_t bsum[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok = blockIdx.x * 8 + warp;
  int cnt = 0;
  if (tok < n) {
    const MaskGeom g = make_geom(n, w, flags, false);
    const int slot = inv[tok];
    const SlotRange r = key_range(g, slot);
    const bool in_frontier = cur[tok] != 0;
    for (int t = lane; t < r.count; t += 32) {
      int ks = r.start + t;
      if (r.wrap) ks = wrap_slot(ks, n);
      else if (ks < 0 || ks >= n) continue;
      const int kt = perm[ks];
      if (visible(g, slot, tok, ks, kt)) {
        ++cnt;
        if (in_frontier) nxt[kt] = 1;
      }
    }
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0 && row_count) row_count[tok] = cnt;
  }
  if (lane == 0) bsum[warp] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long s = 0;
    for (int i = 0; i < 8; ++i) s += (unsigned long long)bsum[i];
    if (s) atomicAdd(nnz, s);
  }
}

__global__ void init_kernel(int n, int src, int32_t* cur, int32_t* nxt,
                            unsigned long long* nnz, int L, int32_t* reach) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    cur[i] = (i == src);
    nxt[i] = 0;
  }
  if (blockIdx.x == 0)
    for (int l = threadIdx.x; l < L; l += blockDim.x) { nnz[l] = 0ull; reach[l] = 0; }
}

// reach[l] = popcount of the next frontier; then clear the old frontier so the two
// buffers can swap roles.
__global__ void count_kernel(int n, const int32_t* __restrict__ nxt, int32_t* __restrict__ old,
                             int32_t* reach) {
  int c = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    c += nxt[i] != 0;
    old[i] = 0;
  }
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(reach, c);
}

}  // namespace

size_t coverage_ws_bytes(int L, int n) {
  (void)L;
  return 2 * (((size_t)n * 4 + 255) / 256 * 256);
}

cudaError_t launch_coverage(int L, int n, int w, uint32_t flags, const int32_t* perm,
                            const int32_t* inv, int src, int64_t* nnz, int32_t* row_count,
                            int32_t* reach, void* ws, cudaStream_t st) {
  int32_t* buf[2];
  buf[0] = (int32_t*)ws;
  buf[1] = (int32_t*)((char*)ws + ((size_t)n * 4 + 255) / 256 * 256);
  const int gb = min((n + 255) / 256, 2048);
  init_kernel<<<gb, 256, 0, st>>>(n, src, buf[0], buf[1], (unsigned long long*)nnz, L, reach);
  bump_launches();
  for (int l = 0; l < L; ++l) {
    layer_kernel<<<(n + 7) / 8, 256, 0, st>>>(
        n, w, flags, perm + (size_t)l * n, inv + (size_t)l * n, buf[l & 1], buf[(l & 1) ^ 1],
        row_count ? row_count + (size_t)l * n : nullptr, (unsigned long long*)nnz + l);
    count_kernel<<<gb, 256, 0, st>>>(n, buf[(l & 1) ^ 1], buf[l & 1], reach + l);
    bump_launches(2);
  }
  return cudaGetLastError();
}

}  // namespace sa
