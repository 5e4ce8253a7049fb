// Permutation generation (Alg. 1 line 1): Philox4x32-10 sort keys, a segmented sort by
// (key, token) with one segment per sequence -- one radix pass on the leading key bits,
// then ranking inside each bucket -- and the inverse written with the permutation.
#include <atomic>

#include "sa_common.cuh"

namespace sa {
namespace {

// Sorting n 64-bit keys that are uniform random bits does not need eight radix passes:
// one pass on the leading bits puts every key into a bucket of about 32 keys, and inside a
// bucket the final place of a key is the number of bucket members that precede it in
// (key, token) order, found by direct counting.  Four launches, no assumption on the bucket
// sizes (an unlucky bucket only costs more comparisons), and the order inside a bucket after
// the scatter does not matter, so the scatter may use atomics and the result is still the
// unique ordering by (key, token).
constexpr int kThreadsPerBlock = 256;
constexpr int kMaxBucketBits = 16;

__host__ __device__ inline int bucket_bits_for(int n) {
  int bits = 0;
  while (bits < kMaxBucketBits && (n >> (bits + 5)) > 0) ++bits;   // about 32 keys per bucket
  return bits;
}

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

__device__ __forceinline__ uint32_t bucket_of(uint64_t key, int bits) {
  return bits ? (uint32_t)(key >> (64 - bits)) : 0u;
}

// keys[b][i] and the size of every bucket.  counts must be zero on entry.
__global__ void keys_kernel(uint32_t seed_lo, uint32_t seed_hi, uint32_t layer, int n, int bits,
                            uint64_t* __restrict__ keys, uint32_t* __restrict__ counts) {
  const int b = blockIdx.y;
  uint32_t* cb = counts + ((size_t)b << bits);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint64_t key = sort_key(seed_lo, seed_hi, layer, b, i);
    keys[(size_t)b * n + i] = key;
    atomicAdd(&cb[bucket_of(key, bits)], 1u);
  }
}

// Exclusive scan of the bucket sizes of one sequence, in place, and a copy that the
// scatter advances.  One block per sequence.
__global__ void __launch_bounds__(kThreadsPerBlock)
scan_kernel(uint32_t* __restrict__ counts, uint32_t* __restrict__ cursor, int nbuckets) {
  __shared__ uint32_t part[kThreadsPerBlock];
  uint32_t* c = counts + (size_t)blockIdx.x * nbuckets;
  uint32_t* cur = cursor + (size_t)blockIdx.x * nbuckets;
  const int per = (nbuckets + kThreadsPerBlock - 1) / kThreadsPerBlock;
  const int lo = threadIdx.x * per, hi = min(lo + per, nbuckets);
  uint32_t s = 0;
  for (int j = lo; j < hi; ++j) s += c[j];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 1; o < kThreadsPerBlock; o <<= 1) {
    const uint32_t add = threadIdx.x >= o ? part[threadIdx.x - o] : 0u;
    __syncthreads();
    part[threadIdx.x] += add;
    __syncthreads();
  }
  uint32_t run = part[threadIdx.x] - s;
  for (int j = lo; j < hi; ++j) {
    const uint32_t v = c[j];
    c[j] = run;
    cur[j] = run;
    run += v;
  }
}

// Every (key, token) into its bucket's range, in arbitrary order inside the range.
__global__ void scatter_kernel(const uint64_t* __restrict__ keys, uint32_t* __restrict__ cursor,
                               uint64_t* __restrict__ bkeys, int32_t* __restrict__ btoks, int n,
                               int bits) {
  const int b = blockIdx.y;
  uint32_t* cur = cursor + ((size_t)b << bits);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint64_t key = keys[(size_t)b * n + i];
    const uint32_t pos = atomicAdd(&cur[bucket_of(key, bits)], 1u);
    bkeys[(size_t)b * n + pos] = key;
    btoks[(size_t)b * n + pos] = i;
  }
}

// Slot of every token: start of its bucket plus the number of bucket members that come
// first in (key, token) order.  Writes perm and its inverse.
__global__ void rank_kernel(const uint64_t* __restrict__ bkeys, const int32_t* __restrict__ btoks,
                            const uint32_t* __restrict__ starts, int32_t* __restrict__ perm,
                            int32_t* __restrict__ inv, int n, int bits) {
  const int b = blockIdx.y;
  const uint64_t* kb = bkeys + (size_t)b * n;
  const int32_t* tb = btoks + (size_t)b * n;
  const uint32_t* st = starts + ((size_t)b << bits);
  const uint32_t nbuckets = 1u << bits;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
    const uint64_t key = kb[e];
    const int32_t tok = tb[e];
    const uint32_t bk = bucket_of(key, bits);
    const uint32_t lo = st[bk], hi = bk + 1 < nbuckets ? st[bk + 1] : (uint32_t)n;
    uint32_t rank = 0;
    for (uint32_t j = lo; j < hi; ++j) {
      const uint64_t kj = kb[j];
      rank += (kj < key) || (kj == key && tb[j] < tok);
    }
    const int32_t pos = (int32_t)(lo + rank);
    perm[(size_t)b * n + pos] = tok;
    inv[(size_t)b * n + tok] = pos;
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
  static std::atomic<unsigned char*> ptrs[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  unsigned char* q = ptrs[dev].load(std::memory_order_acquire);
  if (!q) {
    if (cudaGetSymbolAddress((void**)&q, g_static_scratch) != cudaSuccess) return nullptr;
    ptrs[dev].store(q, std::memory_order_release);
  }
  return q;
}

}  // namespace

size_t make_perm_ws_bytes(int B, int n) {
  const size_t bn = (size_t)B * n;
  const size_t nb = (size_t)B << bucket_bits_for(n);
  return 2 * align_up(bn * 8, 256) + align_up(bn * 4, 256) + 2 * align_up(nb * 4, 256);
}

cudaError_t launch_make_perm(uint64_t seed, uint32_t layer, int B, int n, int32_t* perm,
                             int32_t* inv, void* ws, cudaStream_t st) {
  const size_t bn = (size_t)B * n;
  const int bits = bucket_bits_for(n);
  const size_t nb = (size_t)B << bits;
  char* p = (char*)ws;
  uint64_t* keys = (uint64_t*)p; p += align_up(bn * 8, 256);
  uint64_t* bkeys = (uint64_t*)p; p += align_up(bn * 8, 256);
  int32_t* btoks = (int32_t*)p; p += align_up(bn * 4, 256);
  uint32_t* counts = (uint32_t*)p; p += align_up(nb * 4, 256);
  uint32_t* cursor = (uint32_t*)p;

  cudaError_t e = cudaMemsetAsync(counts, 0, nb * 4, st);   // bucket sizes start at zero
  if (e != cudaSuccess) return e;
  const int kb = min((n + kThreadsPerBlock - 1) / kThreadsPerBlock, 1024);
  keys_kernel<<<dim3(kb, B), kThreadsPerBlock, 0, st>>>((uint32_t)seed, (uint32_t)(seed >> 32),
                                                        layer, n, bits, keys, counts);
  scan_kernel<<<B, kThreadsPerBlock, 0, st>>>(counts, cursor, 1 << bits);
  scatter_kernel<<<dim3(kb, B), kThreadsPerBlock, 0, st>>>(keys, cursor, bkeys, btoks, n, bits);
  rank_kernel<<<dim3(kb, B), kThreadsPerBlock, 0, st>>>(bkeys, btoks, counts, perm, inv, n, bits);
  bump_launches(4);
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
  // Only the bucket counters have to start at zero, and the launcher clears them on the
  // stream itself; the key and token arrays are written in full before anything reads
  // them, so whatever the previous call left behind is never seen.
  return launch_make_perm(seed, layer, B, n, perm, inv, scratch, (cudaStream_t)stream) ==
                 cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
