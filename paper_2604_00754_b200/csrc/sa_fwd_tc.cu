// Fused permuted-window attention forward for sm_100a on the 5th-generation tensor cores.
//
// A persistent grid (one CTA per SM) walks a list of work items.  One item is two 128-row
// query tiles that share one stream of 128-key K/V tiles: two query heads of one GQA group
// over the same 128 slots (group size even), or two adjacent slot tiles of one head
// (otherwise).  Rows of Q, K and V are gathered straight from HBM into 128-byte-swizzled
// shared-memory tiles by TMA gather (four rows per copy, row numbers taken from perm), so
// no permuted copy of any tensor exists.  S = Q K^T and O += P V run as tcgen05.mma with
// fp32 accumulators in tensor memory; the softmax (Eq. 1, with the mask of App. B applied
// per element) runs in registers, one thread per query row, and writes P back to tensor
// memory as the A operand of the second product.  The epilogue normalises, applies the gate
// of Eq. 5 when asked, and scatters each row to its original position.
//
// Warp roles (384 threads): warp 0 TMA producer, warp 1 MMA issuer, warp 2 TMEM
// allocator, warps 4-7 softmax/epilogue of query tile 0, warps 8-11 of query tile 1.
// While one tile's softmax runs, the tensor core works on the other tile.  K and V tiles
// travel through one ring of shared-memory slots (K0 V0 K1 V1 ...), and every barrier is
// addressed by counters that run on across items, so the loads, products and epilogue of
// neighbouring items overlap.
//
// Every mbarrier wait is bounded; on expiry the CTA records SA_ERR_TIMEOUT in the device
// status word, stops issuing work, drains what it started and returns.
#include <cuda.h>

#include "sa_fwd_tc.cuh"

namespace sa {
namespace {

constexpr int kTile = 128;           // query rows per tile and keys per K/V tile
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 2000000000ll;  // about one second

enum TileClass { kSkip = 0, kFull = 1, kCausalOnly = 2, kEdge = 3 };

struct TcParams {
  CUtensorMap tm_q, tm_k, tm_v;
  const int32_t* perm;        // null for the SWA branch
  void* y;
  void* y_branch;
  const void* y_other;
  float* lse;
  const float* gate_logits;
  int* status;
  const int* abort_flag;
  int B, Hq, Hkv, G, n, w, h;
  int causal, linear, one_sided, swa, full_range;
  int pair_heads;             // 1: tiles = two heads, same slots; 0: two slot tiles, one head
  int n_tiles;                // slot tiles of 128
  int items_per_kv;           // work items per (b, hk)
  int total_items;
  float scale2;               // softmax scale * log2(e)
  int64_t q_row_b, q_row_h, q_col_h;    // tensor-map coordinates: row = b*row_b + h*row_h + tok
  int64_t kv_row_b, kv_row_h, kv_col_h;
  int64_t qs[3];              // element strides of y / y_branch / y_other
};

// ----------------------------------------------------------------------------- PTX

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the limit ran out or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* gave_up,
                                          int* status) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*gave_up) return false;
    if (clock64() - t0 > kWaitCycles) {
      *gave_up = 1;
      atomicCAS(status, SA_OK, SA_ERR_TIMEOUT);
      return false;
    }
  }
}

// Four rows of 64 bf16 (128 bytes) each, rows r0..r3 of the 2-D tensor, into 512 bytes of
// 128-byte-swizzled shared memory.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tm, int col, int r0,
                                            int r1, int r2, int r3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc,
                                       uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc,
                                       uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc)
      : "memory");
}

#define SA_R8(v, o) "=r"(v[o]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), \
                    "=r"(v[o + 4]), "=r"(v[o + 5]), "=r"(v[o + 6]), "=r"(v[o + 7])
#define SA_W8(v, o) "r"(v[o]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), \
                    "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7])

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : SA_R8(v, 0), SA_R8(v, 8), SA_R8(v, 16), SA_R8(v, 24)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
      ::SA_W8(v, 0), SA_W8(v, 8), SA_W8(v, 16), SA_W8(v, 24), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::SA_W8(v, 0), SA_W8(v, 8), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// ---------------------------------------------------------------------- descriptors

// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride
// byte offsets in 16-byte units, descriptor version 1 (sm_100), layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes,
                                              uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------- geometry

struct Geo {
  int q0[2];        // first slot of each query tile
  int hq[2];        // query head of each tile
  int valid[2];     // tile exists
  int kstart;       // virtual slot of the first key of K/V tile 0
  int T;            // K/V tiles in the stream
};

__device__ __forceinline__ int tile_class(const TcParams& p, int q0, int kv) {
  const int q1 = q0 + kTile - 1, k1 = kv + kTile - 1;
  if (p.full_range) return kv < p.n ? kEdge : kSkip;
  if (p.one_sided) {
    if (kv > q1 || k1 < q0 - (p.w - 1)) return kSkip;
    if (kv >= 0 && kv >= q1 - (p.w - 1) && k1 <= q0) return kFull;
    return kEdge;
  }
  if (kv > q1 + p.h || k1 < q0 - p.h) return kSkip;
  const bool inside = (k1 - q0 <= p.h) && (q1 - kv <= p.h) &&
                      (!p.linear || (kv >= 0 && k1 < p.n)) && q1 < p.n;
  if (!inside) return kEdge;
  if (!p.causal) return kFull;
  // plain SWA: keys wholly before the queries need no causal test (no wrap inside)
  if (p.swa && kv >= 0 && k1 <= q0) return kFull;
  return kCausalOnly;
}

__device__ __forceinline__ Geo make_geo(const TcParams& p, int item, int hk) {
  Geo g;
  if (p.pair_heads) {
    const int pairs = p.G / 2;
    const int tile = item / pairs, pr = item % pairs;
    g.q0[0] = g.q0[1] = tile * kTile;
    g.hq[0] = hk * p.G + 2 * pr;
    g.hq[1] = g.hq[0] + 1;
    g.valid[0] = g.valid[1] = 1;
  } else {
    const int tpairs = (p.n_tiles + 1) / 2;
    const int tp = item % tpairs, hh = item / tpairs;
    g.q0[0] = 2 * tp * kTile;
    g.q0[1] = g.q0[0] + kTile;
    g.hq[0] = g.hq[1] = hk * p.G + hh;
    g.valid[0] = 1;
    g.valid[1] = g.q0[1] < p.n;
  }
  const int qfirst = g.q0[0];
  const int qlast = min((g.valid[1] ? g.q0[1] : g.q0[0]) + kTile - 1, p.n - 1);
  int kend;
  if (p.full_range) {
    g.kstart = 0;
    kend = p.n - 1;
  } else if (p.one_sided) {
    g.kstart = max(qfirst - (p.w - 1), 0);
    kend = qlast;
  } else if (p.linear) {
    g.kstart = max(qfirst - p.h, 0);
    kend = min(qlast + p.h, p.n - 1);
  } else {
    g.kstart = qfirst - p.h;
    kend = qlast + p.h;
  }
  g.T = (kend - g.kstart + kTile) / kTile;
  return g;
}

__device__ __forceinline__ int actual_slot(const TcParams& p, int v) {
  if (p.full_range || p.linear || p.one_sided) return min(max(v, 0), p.n - 1);
  v %= p.n;
  return v < 0 ? v + p.n : v;
}

// ------------------------------------------------------------------- shared memory

// Ring sizes: kSlots K/V tile slots, kTok key-token lists.  The token list written for K
// tile g is overwritten at tile g + kTok.  To load that tile the producer first has to win
// ring use 2(g + kTok), i.e. see use 2(g + kTok) - kSlots freed.  If that use is V_x it is
// freed by the completion of P V of tile x, which was issued after the softmax of x; if it
// is K_x, by the completion of Q K^T of x, issued after the softmax of x - 1.  The softmax
// of tile g is therefore over when x >= g (odd difference) or x - 1 >= g (even).
template <int D>
struct Cfg {
  static constexpr int kTileBytes = kTile * D * 2;
  static constexpr int kChunks = D / 64;          // 128-byte column blocks per row
  static constexpr int kChunkBytes = kTile * 128;
  static constexpr int kSlots = D == 128 ? 5 : 8;
  static constexpr int kTok = D == 128 ? 4 : 8;
  static_assert((2 * kTok - kSlots) % 2 ? (2 * kTok - kSlots >= 1) : (2 * kTok - kSlots >= 4),
                "token ring too short for the slot ring");
  static constexpr int kOffQ = 0;
  static constexpr int kOffRing = 2 * kTileBytes;
  static constexpr int kOffTok = kOffRing + kSlots * kTileBytes;
  static constexpr int kOffBar = kOffTok + kTok * kTile * 4;
  // mbarriers, 8 bytes each
  static constexpr int kBarQFull = 0, kBarQEmpty = 1, kBarSlotFull = 2,
                       kBarSlotEmpty = kBarSlotFull + kSlots, kBarTokFull = kBarSlotEmpty + kSlots,
                       kBarSFull = kBarTokFull + kTok, kBarPReady = kBarSFull + 2,
                       kBarODone = kBarPReady + 2, kNumBars = kBarODone + 2;
  static constexpr int kOffMisc = kOffBar + kNumBars * 8;   // TMEM base address, gave_up flag
  static constexpr int kBytes = kOffMisc + 16;
  static constexpr uint32_t kColO = 256;                     // O_t at 256 + t*D; S_t at t*128
  static_assert(kBytes <= 232448, "shared memory");
};

// ------------------------------------------------------------------------- kernel

template <int D>
__global__ void __launch_bounds__(kThreads, 1) fwd_tc_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using C = Cfg<D>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (p.abort_flag && *p.abort_flag) return;  // an earlier check rejected perm/inv (uniform)
  // Once any CTA has recorded a timeout the rest of the grid leaves at once instead of
  // each waiting out its own limit.
  if (*(volatile int*)p.status == SA_ERR_TIMEOUT) return;
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                        // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) atomicCAS(p.status, SA_OK, SA_ERR_CUDA);
    return;
  }
  const uint32_t bar0 = sbase + C::kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* gave_up = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);

  if (threadIdx.x == 0) {
    *gave_up = 0;
    for (int i = 0; i < C::kNumBars; ++i)
      mbar_init(bar(i), (i == C::kBarPReady || i == C::kBarPReady + 1) ? kTile : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Registers move from the producer / issuer warps to the softmax warps, which hold a
  // whole score row each.
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    bool ok = true;
    uint32_t use = 0;      // ring uses so far
    uint32_t gt = 0;       // K tiles so far
    uint32_t it = 0;       // items so far
    auto ring_wait = [&](uint32_t u) {
      const uint32_t round = u / C::kSlots;
      bool r = true;
      if (round) r = mbar_wait(bar(C::kBarSlotEmpty + u % C::kSlots), (round - 1) & 1u, gave_up,
                               p.status);
      return (bool)__all_sync(0xffffffffu, r);
    };
    auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, int col0, const int (&rows)[4],
                         uint32_t mb) {
#pragma unroll
      for (int c = 0; c < C::kChunks; ++c)
        tma_gather4(dst + c * C::kChunkBytes + lane * 512, tm, col0 + 64 * c, rows[0], rows[1],
                    rows[2], rows[3], mb);
    };
    for (int w_item = blockIdx.x; w_item < p.total_items && ok; w_item += gridDim.x, ++it) {
      const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
      const int hk = bh % p.Hkv, b = bh / p.Hkv;
      const Geo g = make_geo(p, item, hk);
      const int32_t* perm = p.perm ? p.perm + (size_t)b * p.n : nullptr;
      const int64_t kv_row0 = b * p.kv_row_b + hk * p.kv_row_h;
      const int kv_col0 = (int)(hk * p.kv_col_h);
      for (int j = 0; j < g.T && ok; ++j, ++gt) {
        int rows[4], toks[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int slot = actual_slot(p, g.kstart + j * kTile + 4 * lane + r);
          toks[r] = perm ? perm[slot] : slot;
          rows[r] = (int)(kv_row0 + toks[r]);
        }
        // K_j and the tokens of its keys
        if (!(ok = ring_wait(use))) break;
        {
          const uint32_t mb = bar(C::kBarSlotFull + use % C::kSlots);
          *reinterpret_cast<int4*>(smem + C::kOffTok + (gt % C::kTok) * (kTile * 4) + 16 * lane) =
              make_int4(toks[0], toks[1], toks[2], toks[3]);
          if (lane == 0) mbar_expect_tx(mb, C::kTileBytes);
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C::kBarTokFull + gt % C::kTok));
          load_tile(&p.tm_k, sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes, kv_col0, rows,
                    mb);
          ++use;
        }
        if (j == 0) {
          // Q of this item, once the products of the previous item no longer read it
          if (it) ok = mbar_wait(bar(C::kBarQEmpty), (it - 1) & 1u, gave_up, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) mbar_expect_tx(bar(C::kBarQFull), 2 * C::kTileBytes);
          __syncwarp();
          for (int t = 0; t < 2; ++t) {
            int qrows[4];
            const int64_t row0 = b * p.q_row_b + g.hq[t] * p.q_row_h;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const int slot = min(g.q0[t] + 4 * lane + r, p.n - 1);
              qrows[r] = (int)(row0 + (perm ? perm[slot] : slot));
            }
            load_tile(&p.tm_q, sbase + C::kOffQ + t * C::kTileBytes, (int)(g.hq[t] * p.q_col_h),
                      qrows, bar(C::kBarQFull));
          }
        }
        // V_j
        if (!(ok = ring_wait(use))) break;
        {
          const uint32_t mb = bar(C::kBarSlotFull + use % C::kSlots);
          if (lane == 0) mbar_expect_tx(mb, C::kTileBytes);
          __syncwarp();
          load_tile(&p.tm_v, sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes, kv_col0, rows,
                    mb);
          ++use;
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kTile, kTile, false);
      constexpr uint32_t idesc_pv = instr_desc(kTile, D, true);
      bool ok = true;
      uint32_t use = 0, it = 0;
      uint32_t p_cnt[2] = {0, 0};
      auto slot_addr = [&](uint32_t u) {
        return sbase + C::kOffRing + (u % C::kSlots) * C::kTileBytes;
      };
      auto slot_wait = [&](uint32_t u) {
        return mbar_wait(bar(C::kBarSlotFull + u % C::kSlots), (u / C::kSlots) & 1u, gave_up,
                         p.status);
      };
      auto issue_qk = [&](int t, uint32_t ka) {
        const uint32_t qa = sbase + C::kOffQ + t * C::kTileBytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * C::kChunkBytes + (kk % 4) * 32;
          mma_ss(tmem + t * 128, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024),
                 idesc_qk, kk > 0);
        }
        tc_commit(bar(C::kBarSFull + t));
      };
      for (int w_item = blockIdx.x; w_item < p.total_items && ok; w_item += gridDim.x, ++it) {
        const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
        const Geo g = make_geo(p, item, bh % p.Hkv);
        auto active = [&](int t, int j) {
          return g.valid[t] && j < g.T && tile_class(p, g.q0[t], g.kstart + j * kTile) != kSkip;
        };
        int last[2] = {-1, -1};   // last active K/V tile of each query tile
        for (int t = 0; t < 2; ++t)
          for (int j = g.T - 1; j >= 0; --j)
            if (active(t, j)) { last[t] = j; break; }
        int started[2] = {0, 0};
        // ring uses of this item: K_j = use + 2j, V_j = use + 2j + 1
        ok = mbar_wait(bar(C::kBarQFull), it & 1u, gave_up, p.status);
        if (ok) ok = slot_wait(use);
        if (!ok) break;
        tc_fence_after();
        for (int t = 0; t < 2; ++t)
          if (active(t, 0)) issue_qk(t, slot_addr(use));
        tc_commit(bar(C::kBarSlotEmpty + use % C::kSlots));
        if (g.T == 1) tc_commit(bar(C::kBarQEmpty));
        for (int j = 0; j < g.T && ok; ++j) {
          const uint32_t uv = use + 2 * j + 1, uk = use + 2 * j + 2;
          const bool have_next = j + 1 < g.T;
          bool k_ready = false, v_ready = false;
          for (int t = 0; t < 2 && ok; ++t) {
            if (active(t, j)) {
              if (!v_ready) { ok = slot_wait(uv); v_ready = true; }
              if (ok) ok = mbar_wait(bar(C::kBarPReady + t), p_cnt[t] & 1u, gave_up, p.status);
              if (!ok) break;
              ++p_cnt[t];
              tc_fence_after();
              const uint32_t va = slot_addr(uv);
#pragma unroll
              for (int kk = 0; kk < kTile / 16; ++kk)
                mma_ts(tmem + C::kColO + t * D, tmem + t * 128 + kk * 8,
                       smem_desc(va + kk * 2048, C::kChunkBytes, 1024), idesc_pv,
                       (started[t] | kk) != 0);
              started[t] = 1;
              if (j == last[t]) tc_commit(bar(C::kBarODone + t));
            }
            if (have_next && active(t, j + 1)) {
              if (!k_ready) {
                ok = slot_wait(uk);
                if (!ok) break;
                tc_fence_after();
                k_ready = true;
              }
              issue_qk(t, slot_addr(uk));
            }
          }
          if (ok && !v_ready) ok = slot_wait(uv);
          if (ok && have_next && !k_ready) ok = slot_wait(uk);
          if (!ok) break;
          // the slots free when the products issued so far have finished
          tc_commit(bar(C::kBarSlotEmpty + uv % C::kSlots));
          if (have_next) tc_commit(bar(C::kBarSlotEmpty + uk % C::kSlots));
          if (j + 2 == g.T) tc_commit(bar(C::kBarQEmpty));
        }
        use += 2 * g.T;
      }
    }
    __syncwarp();
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
    // ------------------------------------------------- softmax and epilogue
    const int t = (warp - 4) / 4;
    const int row = threadIdx.x - 128 - t * 128;       // 0..127 == TMEM lane
    const uint32_t lane_addr = (uint32_t)(row & ~31) << 16;
    const uint32_t s_addr = tmem + lane_addr + t * 128;
    const uint32_t o_addr = tmem + lane_addr + C::kColO + t * D;
    uint32_t s_cnt = 0, o_cnt = 0, gt = 0;
    bool ok = true;

    for (int w_item = blockIdx.x; w_item < p.total_items && ok; w_item += gridDim.x) {
      const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
      const int hk = bh % p.Hkv, b = bh / p.Hkv;
      const Geo g = make_geo(p, item, hk);
      const uint32_t gt0 = gt;
      gt += g.T;
      if (!g.valid[t]) continue;
      const int32_t* perm = p.perm ? p.perm + (size_t)b * p.n : nullptr;
      const int qv = g.q0[t] + row;
      const bool row_valid = qv < p.n;
      const int q_tok = row_valid ? (perm ? perm[qv] : qv) : 0;
      const int qcmp = (p.causal && !p.one_sided) ? q_tok : 0x7fffffff;
      float m = -INFINITY, l = 0.f;
      bool started = false;

      for (int j = 0; j < g.T; ++j) {
        const int kv = g.kstart + j * kTile;
        const int cls = tile_class(p, g.q0[t], kv);
        if (cls == kSkip) continue;
        const uint32_t tg = gt0 + j;
        ok = mbar_wait(bar(C::kBarTokFull + tg % C::kTok), (tg / C::kTok) & 1u, gave_up, p.status);
        if (ok) ok = mbar_wait(bar(C::kBarSFull + t), s_cnt & 1u, gave_up, p.status);
        ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below are warp-collective
        if (!ok) break;
        ++s_cnt;
        tc_fence_after();

        uint32_t sr[kTile];
#pragma unroll
        for (int c = 0; c < 4; ++c)
          tmem_ld32(s_addr + 32 * c, reinterpret_cast<uint32_t(&)[32]>(sr[32 * c]));
        tmem_wait_ld();
        const int32_t* ktok = reinterpret_cast<const int32_t*>(smem + C::kOffTok) +
                              (tg % C::kTok) * kTile;
        if (cls == kCausalOnly) {
#pragma unroll
          for (int c = 0; c < kTile; c += 4) {
            const int4 kt = *reinterpret_cast<const int4*>(ktok + c);
            if (kt.x > qcmp) sr[c] = 0xff800000u;
            if (kt.y > qcmp) sr[c + 1] = 0xff800000u;
            if (kt.z > qcmp) sr[c + 2] = 0xff800000u;
            if (kt.w > qcmp) sr[c + 3] = 0xff800000u;
          }
        } else if (cls == kEdge) {
          // visible columns form one interval [lo, hi] of this row, cut by the token order
          int lo, hi;
          if (p.one_sided) { lo = p.full_range ? -kv : qv - (p.w - 1) - kv; hi = qv - kv; }
          else if (p.full_range && !p.linear) { lo = -kv; hi = p.n - 1 - kv; }
          else { lo = qv - p.h - kv; hi = qv + p.h - kv; }
          if (p.linear || p.full_range || p.one_sided) {
            lo = max(lo, -kv);
            hi = min(hi, p.n - 1 - kv);
          }
          if (hi < lo) { lo = 1 << 30; hi = lo; }
          const uint32_t span = (uint32_t)(hi - lo);
#pragma unroll
          for (int c = 0; c < kTile; c += 4) {
            const int4 kt = *reinterpret_cast<const int4*>(ktok + c);
            if ((uint32_t)(c - lo) > span || kt.x > qcmp) sr[c] = 0xff800000u;
            if ((uint32_t)(c + 1 - lo) > span || kt.y > qcmp) sr[c + 1] = 0xff800000u;
            if ((uint32_t)(c + 2 - lo) > span || kt.z > qcmp) sr[c + 2] = 0xff800000u;
            if ((uint32_t)(c + 3 - lo) > span || kt.w > qcmp) sr[c + 3] = 0xff800000u;
          }
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
#pragma unroll
        for (int c = 2; c < kTile; c += 4) {
          mx0 = max3(mx0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
          if (c + 2 < kTile)
            mx1 = max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
        }
        const float m_new = fmaxf(m, fmaxf(mx0, mx1));
        // Lazy rescaling: keep the old reference maximum while the new one is within 2^8.
        const bool grow = (m_new - m) * p.scale2 > 8.f || (m == -INFINITY && m_new > -INFINITY);
        if (!started) {
          m = m_new;
        } else if (__any_sync(0xffffffffu, grow)) {
          const float f = grow ? exp2f((m - m_new) * p.scale2) : 1.f;
          if (grow) { l *= f; m = m_new; }
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t raw[32];
            tmem_ld32(o_addr + 32 * c, raw);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x) raw[x] = __float_as_uint(__uint_as_float(raw[x]) * f);
            tmem_st32(o_addr + 32 * c, raw);
          }
        }
        started = true;
        const float neg = (m == -INFINITY) ? 0.f : -m * p.scale2;
        const float2 sc2 = make_float2(p.scale2, p.scale2), ng2 = make_float2(neg, neg);
        float2 lsum = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            const float2 a = __ffma2_rn(make_float2(__uint_as_float(sr[32 * c + 2 * x]),
                                                    __uint_as_float(sr[32 * c + 2 * x + 1])),
                                        sc2, ng2);
            const float2 e = make_float2(exp2f(a.x), exp2f(a.y));
            lsum = __fadd2_rn(lsum, e);
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(e.x, e.y);
            pk[x] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          tmem_st16(s_addr + 16 * c, pk);
        }
        l += lsum.x + lsum.y;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(C::kBarPReady + t));
      }
      if (!ok) break;

      ok = mbar_wait(bar(C::kBarODone + t), o_cnt & 1u, gave_up, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ++o_cnt;
      tc_fence_after();
      const float inv_l = 1.f / l;
      float g_this = 1.f, g_other = 0.f;
      const int hq = g.hq[t];
      if (p.gate_logits) {
        const float s_sa = 1.f / (1.f + __expf(-p.gate_logits[hq]));
        const float s_swa = 1.f / (1.f + __expf(-p.gate_logits[p.Hq + hq]));
        g_this = p.swa ? s_swa : s_sa;
        g_other = p.swa ? s_sa : s_swa;
      }
      const int64_t off = b * p.qs[0] + hq * p.qs[1] + (int64_t)q_tok * p.qs[2];
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t raw[32];
        tmem_ld32(o_addr + 32 * c, raw);       // warp-collective: every lane takes part
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            float o[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) o[x] = __uint_as_float(raw[8 * x8 + x]) * inv_l;
            const int64_t e = off + 32 * c + 8 * x8;
            if (p.y_branch) {
              uint4 st;
              __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&st);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                h2[x] = __floats2bfloat162_rn(o[2 * x], o[2 * x + 1]);
                o[2 * x] = __low2float(h2[x]);
                o[2 * x + 1] = __high2float(h2[x]);
              }
              *reinterpret_cast<uint4*>((__nv_bfloat16*)p.y_branch + e) = st;
            }
            if (p.gate_logits) {
#pragma unroll
              for (int x = 0; x < 8; ++x) o[x] *= g_this;
              if (p.y_other) {
                const uint4 ot = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)p.y_other + e);
                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&ot);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  o[2 * x] = fmaf(g_other, __low2float(h2[x]), o[2 * x]);
                  o[2 * x + 1] = fmaf(g_other, __high2float(h2[x]), o[2 * x + 1]);
                }
              }
            }
            if (p.y) {
              uint4 st;
              __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&st);
#pragma unroll
              for (int x = 0; x < 4; ++x) h2[x] = __floats2bfloat162_rn(o[2 * x], o[2 * x + 1]);
              *reinterpret_cast<uint4*>((__nv_bfloat16*)p.y + e) = st;
            }
          }
        }
      }
      if (p.lse && row_valid)
        p.lse[((size_t)b * p.Hq + hq) * p.n + q_tok] = (m * p.scale2 + log2f(l)) * kLn2;
      // the next item's first P V overwrites O: order these reads before the arrive that
      // lets it start
      tc_fence_before();
    }
  }

  // ----------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*gave_up && warp == 0 && lane == 0) {
    // Someone ran out of time: give copies that are still in flight a bounded chance to land
    // before the shared memory is released.
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) {}
  }
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------- host

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
            cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

// Coordinates of row (b, h, tok) in a 2-D view [rows, token_stride] of a tensor with element
// strides s[0..2]; false when the layout cannot be viewed that way.
bool row_view(const int64_t s[3], int H, int d, int64_t* row_b, int64_t* row_h, int64_t* col_h) {
  const int64_t ts = s[2];
  if (ts < d || s[0] % ts != 0) return false;
  *row_b = s[0] / ts;
  if (s[1] % ts == 0) {
    *row_h = s[1] / ts;
    *col_h = 0;
  } else {
    if (s[1] * (H - 1) + d > ts) return false;
    *row_h = 0;
    *col_h = s[1];
  }
  return true;
}

bool make_map(CUtensorMap* tm, const void* base, int64_t ts, int64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rows <= 0 || rows > 0x7fffffffll) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)ts, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ts * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_disabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("SA_DISABLE_TC");
    v = (e && e[0] == '1') ? 1 : 0;
  }
  return v == 1;
}

}  // namespace

bool tc_forward_supported(const FwdArgs& a, int dtype) {
  if (tc_disabled() || dtype != SA_BF16 || (a.d != 128 && a.d != 64)) return false;
  if (a.n < 1 || (int64_t)a.B * a.Hq * ((a.n + kTile - 1) / kTile) > 0x3fffffff) return false;
  int64_t rb, rh, ch;
  if (!row_view(a.qs, a.Hq, a.d, &rb, &rh, &ch)) return false;
  if (!row_view(a.ks, a.Hkv, a.d, &rb, &rh, &ch)) return false;
  if (a.qs[2] > (1 << 20) || a.ks[2] > (1 << 20)) return false;
  return encode_fn() != nullptr;
}

cudaError_t launch_fwd_tc(const FwdArgs& a, cudaStream_t st) {
  TcParams p{};
  int64_t rb, rh, ch;
  row_view(a.qs, a.Hq, a.d, &rb, &rh, &ch);
  p.q_row_b = rb; p.q_row_h = rh; p.q_col_h = ch;
  const int64_t q_rows = (a.B - 1) * rb + (a.Hq - 1) * rh + a.n;
  row_view(a.ks, a.Hkv, a.d, &rb, &rh, &ch);
  p.kv_row_b = rb; p.kv_row_h = rh; p.kv_col_h = ch;
  const int64_t kv_rows = (a.B - 1) * rb + (a.Hkv - 1) * rh + a.n;
  if (!make_map(&p.tm_q, a.q, a.qs[2], q_rows) || !make_map(&p.tm_k, a.k, a.ks[2], kv_rows) ||
      !make_map(&p.tm_v, a.v, a.ks[2], kv_rows))
    return cudaErrorInvalidValue;
  p.perm = a.swa ? nullptr : a.perm;
  p.y = a.y; p.y_branch = a.y_branch; p.y_other = a.y_other; p.lse = a.lse;
  p.gate_logits = a.gate_logits;
  p.status = status_ptr();
  if (!p.status) return cudaErrorUnknown;
  p.abort_flag = a.abort_flag;
  p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.Hq / a.Hkv; p.n = a.n; p.w = a.w;
  const MaskGeom mg = make_geom(a.n, a.w, a.flags, a.swa);
  p.h = mg.h;
  p.causal = mg.causal; p.linear = mg.linear; p.one_sided = mg.one_sided; p.swa = a.swa;
  p.full_range = mg.one_sided ? (a.w - 1 >= a.n) : (2ll * mg.h + 1 >= a.n);
  p.pair_heads = (p.G % 2 == 0);
  p.n_tiles = (a.n + kTile - 1) / kTile;
  p.items_per_kv = p.pair_heads ? p.n_tiles * (p.G / 2) : ((p.n_tiles + 1) / 2) * p.G;
  p.scale2 = a.scale * kLog2e;
  for (int i = 0; i < 3; ++i) p.qs[i] = a.qs[i];
  p.total_items = a.B * a.Hkv * p.items_per_kv;

  static int sm_count[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= 64) return e != cudaSuccess ? e : cudaErrorInvalidDevice;
  if (!sm_count[dev]) {
    e = cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  const unsigned grid = (unsigned)min(p.total_items, sm_count[dev]);
  if (a.d == 128) {
    const int smem = Cfg<128>::kBytes;
    e = cudaFuncSetAttribute(fwd_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    fwd_tc_kernel<128><<<grid, kThreads, smem, st>>>(p);
  } else {
    const int smem = Cfg<64>::kBytes;
    e = cudaFuncSetAttribute(fwd_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    fwd_tc_kernel<64><<<grid, kThreads, smem, st>>>(p);
  }
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa
