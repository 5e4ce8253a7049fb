// Permutation generation (Alg. 1 line 1): Philox4x32-10 sort keys, a segmented
// least-significant-digit radix sort (8 passes of 8 bits over 64-bit keys, one segment
// per sequence), and the inverse by scatter, fused into the last pass.
//
// The radix sort is stable, so equal keys keep increasing token order: the result is
// the unique ordering by (key, token).
#include "sa_common.cuh"

namespace sa {
namespace {

constexpr int kRadixBits = 8;
constexpr int kRadix = 1 << kRadixBits;
constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kItems = 8;                          // keys per thread per tile
constexpr int kTile = kSortThreads * kItems;       // keys per block
constexpr int kPasses = 64 / kRadixBits;

__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
  const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
  const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
  const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
  c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

// Philox4x32 with 10 rounds (Salmon et al., SC'11); the key follows a Weyl sequence.
__device__ __forceinline__ uint64_t sort_key(uint32_t seed_lo, uint32_t seed_hi, uint32_t layer,
                                             uint32_t b, uint32_t i) {
  uint32_t c[4] = {i, b, layer, 0u};
  uint32_t k0 = seed_lo, k1 = seed_hi;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    philox_round(c, k0, k1);
  }
  return ((uint64_t)c[0] << 32) | c[1];
}

__global__ void keys_kernel(uint32_t seed_lo, uint32_t seed_hi, uint32_t layer, int n,
                            uint64_t* __restrict__ keys, int32_t* __restrict__ vals) {
  const int b = blockIdx.y;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    keys[(size_t)b * n + i] = sort_key(seed_lo, seed_hi, layer, b, i);
    vals[(size_t)b * n + i] = i;
  }
}

// counts[b][digit][blk] = number of keys of tile blk of sequence b with that digit.
__global__ void __launch_bounds__(kSortThreads)
hist_kernel(const uint64_t* __restrict__ keys, int n, int shift, int nblk,
            uint32_t* __restrict__ counts) {
  __shared__ uint32_t h[kRadix];
  const int b = blockIdx.y, blk = blockIdx.x;
  h[threadIdx.x] = 0;
  __syncthreads();
  const uint64_t* kb = keys + (size_t)b * n;
  const int base = blk * kTile;
#pragma unroll
  for (int it = 0; it < kItems; ++it) {
    const int i = base + it * kSortThreads + threadIdx.x;
    if (i < n) atomicAdd(&h[(uint32_t)(kb[i] >> shift) & (kRadix - 1)], 1u);
  }
  __syncthreads();
  counts[((size_t)b * kRadix + threadIdx.x) * nblk + blk] = h[threadIdx.x];
}

// Exclusive scan of counts[b][digit][blk] in (digit, blk) order, in place.  One block per b.
__global__ void __launch_bounds__(kRadix)
scan_kernel(uint32_t* __restrict__ counts, int nblk) {
  __shared__ uint32_t tot[kRadix];
  uint32_t* c = counts + (size_t)blockIdx.x * kRadix * nblk + (size_t)threadIdx.x * nblk;
  uint32_t s = 0;
  for (int j = 0; j < nblk; ++j) s += c[j];
  tot[threadIdx.x] = s;
  __syncthreads();
  // Hillis-Steele inclusive scan over the 256 digit totals
  for (int o = 1; o < kRadix; o <<= 1) {
    const uint32_t add = threadIdx.x >= o ? tot[threadIdx.x - o] : 0u;
    __syncthreads();
    tot[threadIdx.x] += add;
    __syncthreads();
  }
  uint32_t run = tot[threadIdx.x] - s;  // exclusive start of this digit
  for (int j = 0; j < nblk; ++j) {
    const uint32_t v = c[j];
    c[j] = run;
    run += v;
  }
}

// Stable scatter of one tile.  Keys are taken 256 at a time in index order; inside a
// group, a key's rank among equal digits is (equal digits in earlier warps) + (equal
// digits in lower lanes of its own warp).  With `last`, the sorted token list IS perm and
// the inverse is written in the same pass.
__global__ void __launch_bounds__(kSortThreads)
scatter_kernel(const uint64_t* __restrict__ keys_in, const int32_t* __restrict__ vals_in,
               uint64_t* __restrict__ keys_out, int32_t* __restrict__ vals_out,
               int32_t* __restrict__ inv_out, int n, int shift, int nblk,
               const uint32_t* __restrict__ offsets, int last) {
  __shared__ uint32_t base[kRadix];
  __shared__ uint32_t whist[kSortWarps][kRadix];
  const int b = blockIdx.y, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  base[threadIdx.x] = offsets[((size_t)b * kRadix + threadIdx.x) * nblk + blk];
  const uint64_t* kb = keys_in + (size_t)b * n;
  const int32_t* vb = vals_in + (size_t)b * n;
  for (int it = 0; it < kItems; ++it) {
    for (int x = threadIdx.x; x < kSortWarps * kRadix; x += kSortThreads) (&whist[0][0])[x] = 0;
    __syncthreads();
    const int i = blk * kTile + it * kSortThreads + threadIdx.x;
    const bool live = i < n;
    uint64_t key = 0;
    int32_t val = 0;
    uint32_t digit = 0, rank = 0;
    if (live) { key = kb[i]; val = vb[i]; digit = (uint32_t)(key >> shift) & (kRadix - 1); }
    // dead lanes get a private pseudo-digit so they never match a live one
    const uint32_t peers = __match_any_sync(0xffffffffu, live ? digit : (kRadix + lane));
    if (live) {
      rank = __popc(peers & ((1u << lane) - 1u));
      if (rank == 0) whist[warp][digit] = __popc(peers);
    }
    __syncthreads();
    uint32_t pos = 0;
    if (live) {
      pos = base[digit] + rank;
      for (int wv = 0; wv < warp; ++wv) pos += whist[wv][digit];
    }
    __syncthreads();
    {  // advance the running base of digit threadIdx.x past this group
      uint32_t add = 0;
#pragma unroll
      for (int wv = 0; wv < kSortWarps; ++wv) add += whist[wv][threadIdx.x];
      base[threadIdx.x] += add;
    }
    if (live) {
      if (last) {
        vals_out[(size_t)b * n + pos] = val;
        inv_out[(size_t)b * n + val] = (int32_t)pos;
      } else {
        keys_out[(size_t)b * n + pos] = key;
        vals_out[(size_t)b * n + pos] = val;
      }
    }
    __syncthreads();
  }
}

__global__ void validate_perm_kernel(const int32_t* __restrict__ perm,
                                     const int32_t* __restrict__ inv, int n, int* status) {
  const int b = blockIdx.y;
  for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < n; p += gridDim.x * blockDim.x) {
    const int32_t t = perm[(size_t)b * n + p];
    bool ok = t >= 0 && t < n;
    if (ok) ok = inv[(size_t)b * n + t] == p;
    if (!ok) atomicCAS(status, SA_OK, SA_ERR_BAD_PERM);
  }
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Built-in scratch of sa_make_perm_static: part of the library image, so every GPU that
// loads the library holds these bytes until the process exits.  In host code this name is
// only a host-side stand-in for the symbol, never a device address: the launcher below
// resolves the real address with cudaGetSymbolAddress and hands that to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[SA_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, resolved once per device.
unsigned char* static_scratch_ptr() {
  static unsigned char* ptrs[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ptrs[dev]) {
    unsigned char* q = nullptr;
    if (cudaGetSymbolAddress((void**)&q, g_static_scratch) != cudaSuccess) return nullptr;
    ptrs[dev] = q;
  }
  return ptrs[dev];
}

}  // namespace

size_t make_perm_ws_bytes(int B, int n) {
  const size_t bn = (size_t)B * n;
  const int nblk = (n + kTile - 1) / kTile;
  return 2 * align_up(bn * 8, 256) + 2 * align_up(bn * 4, 256) +
         align_up((size_t)B * kRadix * nblk * 4, 256);
}

cudaError_t launch_make_perm(uint64_t seed, uint32_t layer, int B, int n, int32_t* perm,
                             int32_t* inv, void* ws, cudaStream_t st) {
  const size_t bn = (size_t)B * n;
  const int nblk = (n + kTile - 1) / kTile;
  char* p = (char*)ws;
  uint64_t* keys[2];
  int32_t* vals[2];
  keys[0] = (uint64_t*)p; p += align_up(bn * 8, 256);
  keys[1] = (uint64_t*)p; p += align_up(bn * 8, 256);
  vals[0] = (int32_t*)p; p += align_up(bn * 4, 256);
  vals[1] = (int32_t*)p; p += align_up(bn * 4, 256);
  uint32_t* counts = (uint32_t*)p;

  const int kb = min((n + 255) / 256, 1024);
  keys_kernel<<<dim3(kb, B), 256, 0, st>>>((uint32_t)seed, (uint32_t)(seed >> 32), layer, n,
                                           keys[0], vals[0]);
  bump_launches();
  int cur = 0;
  for (int pass = 0; pass < kPasses; ++pass) {
    const int shift = pass * kRadixBits;
    const int last = pass == kPasses - 1;
    hist_kernel<<<dim3(nblk, B), kSortThreads, 0, st>>>(keys[cur], n, shift, nblk, counts);
    scan_kernel<<<B, kRadix, 0, st>>>(counts, nblk);
    scatter_kernel<<<dim3(nblk, B), kSortThreads, 0, st>>>(
        keys[cur], vals[cur], keys[cur ^ 1], last ? perm : vals[cur ^ 1], inv, n, shift, nblk,
        counts, last);
    bump_launches(3);
    cur ^= 1;
  }
  return cudaGetLastError();
}

cudaError_t launch_validate_perm(const int32_t* perm, const int32_t* inv, int B, int n,
                                 cudaStream_t st) {
  int* status = status_ptr();
  if (!status) return cudaErrorUnknown;
  const int kb = min((n + 255) / 256, 1024);
  validate_perm_kernel<<<dim3(kb, B), 256, 0, st>>>(perm, inv, n, status);
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa

extern "C" sa_status sa_make_perm_static(uint64_t seed, uint32_t layer, int32_t B, int32_t n,
                                         int32_t* perm, int32_t* inv, sa_stream_t stream) {
  using namespace sa;
  if (B < 1 || n < 1) return SA_ERR_INVALID_ARG;
  if (B > 32767 || n > (1 << 30)) return SA_ERR_UNSUPPORTED;
  if (!perm || !inv || ((uintptr_t)perm & 15u) || ((uintptr_t)inv & 15u)) return SA_ERR_INVALID_ARG;
  if (make_perm_ws_bytes(B, n) > (size_t)SA_STATIC_SCRATCH_BYTES) return SA_ERR_TOO_LARGE;
  unsigned char* scratch = static_scratch_ptr();
  if (!scratch) return SA_ERR_CUDA;
  // Nothing in the scratch has to start at zero: the key, index and histogram arrays of a
  // call are each written in full by that call before anything reads them, so whatever
  // the previous call left behind is never seen.
  return launch_make_perm(seed, layer, B, n, perm, inv, scratch, (cudaStream_t)stream) ==
                 cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
