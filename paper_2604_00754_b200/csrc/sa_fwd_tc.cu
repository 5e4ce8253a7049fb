// Fused permuted-window attention forward for sm_100a on the 5th-generation tensor cores.
//
// A persistent grid (one CTA per SM) walks a list of work items.  One item is two 128-row
// query tiles that share one stream of 128-key K/V tiles: two query heads of one GQA group
// over the same 128 slots (group size even), or two adjacent slot tiles of one head
// (otherwise).  Rows of Q, K and V are gathered straight from HBM into 128-byte-swizzled
// shared-memory tiles with 16-byte cp.async copies (row numbers taken from perm, the swizzle
// applied in the destination address), so no permuted copy of any tensor exists.  (TMA row
// gather, four rows per copy, measured about 70 cycles per copy per SM on this part, a
// quarter of what the tensor core consumes; the cp.async path is not issue-bound.)  S = Q K^T and O += P V run as tcgen05.mma with
// fp32 accumulators in tensor memory; the softmax (Eq. 1, with the mask of App. B applied
// per element) runs in registers, one thread per query row, and writes P back to tensor
// memory as the A operand of the second product.  The epilogue normalises, applies the gate
// of Eq. 5 when asked, and scatters each row to its original position.
//
// Warp roles (384 threads): warp 0 MMA issuer and TMEM allocator, warps 1-3 gather
// producers (for the one-sided SWA branch, whose rows are consecutive, one thread that loads
// whole tiles by TMA instead), warps 4-7 softmax/epilogue of query tile 0, warps 8-11 of
// query tile 1.
// While one tile's softmax runs, the tensor core works on the other tile.  K and V tiles
// travel through one ring of shared-memory slots (K0 V0 K1 V1 ...), and every barrier is
// addressed by counters that run on across items, so the loads, products and epilogue of
// neighbouring items overlap.
//
// Every mbarrier wait is bounded; on expiry the CTA records SA_ERR_TIMEOUT in the device
// status word, stops issuing work, drains what it started and returns.
#include <type_traits>

#include "sa_fwd_tc.cuh"
#include "sa_gemm_common.cuh"
#include "sa_tc_common.cuh"

namespace sa {
namespace {

constexpr int kTile = 128;           // query rows per tile and keys per K/V tile
constexpr int kThreads = 384;
constexpr int kProducers = 96;       // threads of the three gather warps
constexpr uint32_t kTmemCols = 512;

enum TileClass { kSkip = 0, kFull = 1, kCausalOnly = 2, kEdge = 3 };

struct TcParams {
  const void *q, *k, *v;
  const int32_t* perm;        // null for the SWA branch
  const float *rope_cos, *rope_sin;   // null, or [n, D/2] each: rotate Q and K rows on the way in
  void* y;
  void* y_branch;
  const void* y_other;
  float* lse;
  const float* gate_logits;
  int* status;
  const int* abort_flag;
  int B, Hq, Hkv, G, n, w, h;
  int causal, linear, one_sided, swa, full_range;
  // One-sided SWA branch: whole tiles come by TMA through rank-4 maps (d, token, head, batch)
  int use_tma;
  int pair_heads;             // 1: tiles = two heads, same slots; 0: two slot tiles, one head
  int n_tiles;                // slot tiles of 128
  int items_per_kv;           // work items per (b, hk)
  int total_items;
  float scale2;               // softmax scale * log2(e)
  int64_t qs[3];              // element strides of q / y / y_branch / y_other: batch, head, token
  int64_t ks[3];              // element strides of k / v
};

// ------------------------------------------------------------------------- geometry

struct Geo {
  int q0[2];        // first slot of each query tile
  int hq[2];        // query head of each tile
  int valid[2];     // tile exists
  int kstart;       // virtual slot of the first key of K/V tile 0
  int T;            // K/V tiles in the stream
};

// How the keys [kv, kv + kw) relate to the queries [q0, q0 + 128): not needed at all, all
// visible, visible up to the token order only, or to be tested element by element.
__device__ __forceinline__ int tile_class(const TcParams& p, int q0, int kv, int kw) {
  const int q1 = q0 + kTile - 1, k1 = kv + kw - 1;
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

// The score blocks h (keys kstart + (h << shift) and the 2^shift - 1 after it) that tile_class does not skip for the
// query tile at q0: a contiguous range [first, last], empty (first > last) for a tile
// that does not exist.
__device__ __forceinline__ void active_halves(const TcParams& p, int q0, int valid, int kstart,
                                              int H, int shift, int* first, int* last) {
  const int q1 = q0 + kTile - 1;
  int lo, hi;   // keys of interest: some key of the half >= lo, its first key <= hi
  if (p.full_range) { lo = 0; hi = p.n - 1; }
  else if (p.one_sided) { lo = q0 - (p.w - 1); hi = q1; }
  else { lo = q0 - p.h; hi = q1 + p.h; }
  const int f = max(0, (lo - kstart) >> shift), l = min(H - 1, (hi - kstart) >> shift);
  *first = valid ? f : (1 << 30);
  *last = valid ? l : -1;
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
  static constexpr int kChunkBytes = kTile * 128;
  static constexpr int kSlots = D == 128 ? 5 : 8;
  static constexpr int kTok = D == 128 ? 3 : 8;
  static_assert((2 * kTok - kSlots) % 2 ? (2 * kTok - kSlots >= 1) : (2 * kTok - kSlots >= 4),
                "token ring too short for the slot ring");
  // Q buffers (two query tiles each).  With two (d = 64 leaves the room) the next item's Q is
  // gathered, and its first scores are issued, while the row threads still finish this item:
  // short items (narrow windows) otherwise idle a quarter of their time at every item start.
  static constexpr int kQBufs = D == 128 ? 1 : 2;
  static constexpr int kOffQ = 0;
  static constexpr int kOffRing = kQBufs * 2 * kTileBytes;
  static constexpr int kOffTok = kOffRing + kSlots * kTileBytes;
  static constexpr int kOffQTok = kOffTok + kTok * kTile * 4;   // tokens of the two query tiles
  static constexpr int kOffBar = kOffQTok + 2 * kTile * 4;
  // mbarriers, 8 bytes each
  static constexpr int kBarQFull = 0, kBarQEmpty = kQBufs, kBarSlotFull = 2 * kQBufs,
                       kBarSlotEmpty = kBarSlotFull + kSlots, kBarTokFull = kBarSlotEmpty + kSlots,
                       kBarSFull = kBarTokFull + kTok, kBarPReady = kBarSFull + 4,
                       kBarPvDone = kBarPReady + 4, kBarODone = kBarPvDone + 2,
                       kBarRowsDone = kBarODone + 2, kBarRowsTaken = kBarRowsDone + 2,
                       kNumBars = kBarRowsTaken + 2;
  static constexpr int kOffMisc = kOffBar + kNumBars * 8;   // TMEM base address, gave_up flag
  static constexpr int kBytes = kOffMisc + 16;
  static constexpr uint32_t kColO = 256;                     // O_t at 256 + t*D; S_t at t*128
  static_assert(kBytes <= 232448, "shared memory");
};

// ------------------------------------------------------------------------- kernel

// D: head dimension.  KB: keys per score block, 64 or 128.  With 64 a tile's S columns hold
// two blocks and the scores run two blocks ahead of the softmax; with 128 a block is the
// whole K/V tile and the next scores of a tile follow its P V.
// TMA: the instantiation for launches whose tiles come by TMA (p.use_tma).
// ROPE: the gather producers rotate the rows of Q and K by their tokens' angles (rotary
// position embedding with ORIGINAL positions, Sec. 4.2 / App. B) after the copies have landed.
// COMBINE: the epilogue reads the other branch's finished rows and applies the gates of Eq. 5
// (the instantiation of the launch that closes a gated forward); without it the kernel
// carries no gate code at all.
template <int D, int KB, bool TMA, bool ROPE = false, bool COMBINE = false>
__global__ void __launch_bounds__(kThreads, 1)
fwd_tc_kernel(const __grid_constant__ TcParams p, const __grid_constant__ CUtensorMap tm_q,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using C = Cfg<D>;
  constexpr int kHalf = KB;             // keys per score block
  constexpr int NB = kTile / KB;        // score blocks per K/V tile = S buffers per query tile
  constexpr int kShift = KB == 64 ? 6 : 7;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

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
    note_skip(reinterpret_cast<volatile int*>(smem + C::kOffMisc + 8), p.status, p.abort_flag);
    for (int i = 0; i < C::kNumBars; ++i)
      mbar_init(bar(i), i >= C::kBarRowsTaken ? 64      // the two combining warps
                        : ((i >= C::kBarPReady && i < C::kBarPvDone) || i >= C::kBarRowsDone) ? kTile
                        : (i < C::kBarQEmpty || (i >= C::kBarSlotFull && i < C::kBarSlotEmpty))
                            ? (p.use_tma ? 1 : kProducers) : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  SA_LEAVE_IF_SKIPPED(reinterpret_cast<volatile int*>(smem + C::kOffMisc + 8), 0, tmem, kTmemCols)

  // Registers move from the producer / issuer warps to the softmax warps, which hold a
  // whole score row each.
  if (warp < 4) {
  // Registers per lane over the 12 warps: 4 x 56 + 8 x 224 = 2016, all that the launch holds
  // (12 x 168).  The four warps of a warpgroup must ask for the same count, so the issuing
  // warp and the producer warps go down together.  With 224 registers the 128 scores and the
  // 32 packed probabilities of a softmax thread stay in registers (at 208 they spilled).
  // With ROPE the producers need room for the rotation: 4 x 72 + 8 x 216 = 2016 again.  (The
  // sum may never exceed what the launch holds: a warpgroup asking for more waits for ever.)
  static_assert(4 * 72 + 8 * 216 == 12 * 168 && 4 * 56 + 8 * 224 == 12 * 168, "register split");
  if (ROPE) asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
  else asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
  if (warp >= 1 && TMA) {
    // ------------------------------------------- tile loads by TMA (one thread of warp 1)
    // Rows are consecutive tokens here, so a tile is D / 64 boxes of 128 tokens x 64 columns
    // that the TMA unit lays out in the same swizzled form the gather produces; no producer
    // instructions compete with the softmax warps.  The token index is a dimension of the
    // map, so rows past the sequence are filled with zeros (never with whatever follows in
    // memory, which could be NaN and would poison P V through 0 * NaN); the window mask
    // does not let them count and their outputs are not stored.  The key-token lists are
    // not written: the one-sided rule tests slots only.
    if (threadIdx.x == 32) {
      uint32_t use = 0, gt = 0, it = 0, q_armed = 0xffffffffu;
      bool live = true;
      auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, int tok, int head, int b,
                           uint32_t mb) {
#pragma unroll
        for (int c = 0; c < D / 64; ++c)
          tma_load_4d(dst + c * C::kChunkBytes, tm, 64 * c, tok, head, b, mb);
      };
      for (int w_item = blockIdx.x; w_item < p.total_items && live; w_item += gridDim.x, ++it) {
        const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
        const int hk = bh % p.Hkv, b = bh / p.Hkv;
        const Geo g = make_geo(p, item, hk);
        for (int j = 0; j < g.T; ++j, ++gt) {
          if (use >= (uint32_t)C::kSlots)
            live = mbar_wait(bar(C::kBarSlotEmpty + use % C::kSlots), (use / C::kSlots - 1) & 1u,
                             gave_up, p.status);
          if (!live) break;
          mbar_arrive(bar(C::kBarTokFull + gt % C::kTok));
          uint32_t mb = bar(C::kBarSlotFull + use % C::kSlots);
          mbar_expect_tx(mb, C::kTileBytes);
          load_tile(&tm_k, sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes,
                    g.kstart + j * kTile, hk, b, mb);
          ++use;
          if (j == 0) {
            const uint32_t qb = it % C::kQBufs;
            if (it >= (uint32_t)C::kQBufs)
              live = mbar_wait(bar(C::kBarQEmpty + qb), (it / C::kQBufs - 1) & 1u, gave_up, p.status);
            if (!live) break;
            mbar_expect_tx(bar(C::kBarQFull + qb), 2 * C::kTileBytes);
            q_armed = it;
#pragma unroll
            for (int t = 0; t < 2; ++t)
              load_tile(&tm_q, sbase + C::kOffQ + (2 * qb + t) * C::kTileBytes, g.q0[t], g.hq[t], b,
                        bar(C::kBarQFull + qb));
          }
          if (use >= (uint32_t)C::kSlots)
            live = mbar_wait(bar(C::kBarSlotEmpty + use % C::kSlots), (use / C::kSlots - 1) & 1u,
                             gave_up, p.status);
          if (!live) break;
          mb = bar(C::kBarSlotFull + use % C::kSlots);
          mbar_expect_tx(mb, C::kTileBytes);
          load_tile(&tm_v, sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes,
                    g.kstart + j * kTile, hk, b, mb);
          ++use;
        }
      }
      // loads that were started but never consumed (only after a failed wait) must land
      // before the shared memory goes away: wait for them, again with a limit
      if (!live || *gave_up) {
        const uint32_t first = use > (uint32_t)C::kSlots ? use - C::kSlots : 0u;
        for (uint32_t u = first; u < use; ++u)
          for (int tries = 0; tries < 100000; ++tries) {
            if (mbar_try(bar(C::kBarSlotFull + u % C::kSlots), (u / C::kSlots) & 1u)) break;
            __nanosleep(100);
          }
        if (q_armed != 0xffffffffu)
          for (int tries = 0; tries < 100000; ++tries) {
            if (mbar_try(bar(C::kBarQFull + q_armed % C::kQBufs), (q_armed / C::kQBufs) & 1u)) break;
            __nanosleep(100);
          }
      }
    } else if (COMBINE && warp >= 2) {
      // ------------------------------- gated combine by the two idle warps (Eq. 5)
      // With tiles coming by TMA, warps 2 and 3 have nothing to load.  The row threads store
      // this branch's finished rows ungated (to y_branch, else to y) and arrive on "rows
      // done"; these 64 threads then read them back together with the other branch's rows
      // (both from L2), apply the two gates and write y, 16 bytes per thread and step, off
      // the row threads' path.  Each 16-byte piece is read and written by one thread, so y
      // may be the buffer this branch's rows were stored in.  "Rows taken" tells the row
      // threads that their previous arrival has been seen, so that the two barriers can
      // never be a whole phase apart (a one-bit parity could not tell).
      constexpr int kCpr = D / 8, kRowsPerPass = 64 / kCpr;
      const int ctid = threadIdx.x - 64, chunk = ctid % kCpr, rsub = ctid / kCpr;
      const __nv_bfloat16* mine = (const __nv_bfloat16*)(p.y_branch ? p.y_branch : p.y);
      const __nv_bfloat16* other = (const __nv_bfloat16*)p.y_other;
      __nv_bfloat16* yout = (__nv_bfloat16*)p.y;
      uint32_t done0 = 0, done1 = 0;
      bool live = true;
      for (int w_item = blockIdx.x; w_item < p.total_items && live; w_item += gridDim.x) {
        const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
        const int b = bh / p.Hkv;
        const Geo g = make_geo(p, item, bh % p.Hkv);
        // the other branch's rows of this item will be wanted a whole item from now: start
        // bringing them into L2 (one 128-byte line per thread and step)
#pragma unroll 1
        for (int t = 0; t < 2; ++t) {
          if (!g.valid[t]) continue;
          const __nv_bfloat16* ob = other + b * p.qs[0] + g.hq[t] * p.qs[1];
          for (int x = ctid; x < kTile * (D / 64); x += 64) {
            const int slot = g.q0[t] + x / (D / 64);
            if (slot < p.n)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(ob + (int64_t)slot * p.qs[2] + 64 * (x % (D / 64))));
          }
        }
#pragma unroll 1
        for (int t = 0; t < 2 && live; ++t) {
          if (!g.valid[t]) continue;
          live = mbar_wait(bar(C::kBarRowsDone + t), (t ? done1 : done0) & 1u, gave_up, p.status);
          if (!live) break;
          mbar_arrive(bar(C::kBarRowsTaken + t));
          done0 += 1 - t;
          done1 += t;
          const int hq = g.hq[t];
          const float g_sa = 1.f / (1.f + __expf(-p.gate_logits[hq]));
          const float g_swa = 1.f / (1.f + __expf(-p.gate_logits[p.Hq + hq]));
          const float g_mine = p.swa ? g_swa : g_sa, g_oth = p.swa ? g_sa : g_swa;
          const int64_t base = b * p.qs[0] + hq * p.qs[1] + chunk * 8;
#pragma unroll 1
          for (int r0 = rsub; r0 < kTile; r0 += 4 * kRowsPerPass) {
            uint4 a[4], c4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int slot = g.q0[t] + r0 + u * kRowsPerPass;   // this branch: token == slot
              if (slot < p.n) {
                const int64_t off = base + (int64_t)slot * p.qs[2];
                a[u] = __ldcg(reinterpret_cast<const uint4*>(mine + off));
                c4[u] = __ldcg(reinterpret_cast<const uint4*>(other + off));
              }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int slot = g.q0[t] + r0 + u * kRowsPerPass;
              if (slot < p.n) {
                const __nv_bfloat162* hm = reinterpret_cast<const __nv_bfloat162*>(&a[u]);
                const __nv_bfloat162* ho = reinterpret_cast<const __nv_bfloat162*>(&c4[u]);
                uint4 o;
                __nv_bfloat162* hr = reinterpret_cast<__nv_bfloat162*>(&o);
                // sa term times its gate first, then the local term by fma
                const float gs = p.swa ? g_oth : g_mine, gl = p.swa ? g_mine : g_oth;
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  const __nv_bfloat162 sa2 = p.swa ? ho[x] : hm[x], lo2 = p.swa ? hm[x] : ho[x];
                  hr[x] = __floats2bfloat162_rn(
                      fmaf(gl, __low2float(lo2), gs * __low2float(sa2)),
                      fmaf(gl, __high2float(lo2), gs * __high2float(sa2)));
                }
                *reinterpret_cast<uint4*>(yout + base + (int64_t)slot * p.qs[2]) = o;
              }
            }
          }
        }
      }
    }
  } else if (warp >= 1 && !TMA) {
    // ---------------------------------------------------- gather producers (warps 1-3)
    // Each 16-byte piece of a row goes from global memory to its swizzled place in shared
    // memory with cp.async; one warp instruction moves kRpi whole rows.
    constexpr int kCpr = D / 8;            // 16-byte pieces per row
    constexpr int kRpi = 32 / kCpr;        // rows per warp instruction
    const int ptid = threadIdx.x - 32;     // 0..95
    const int sub = lane / kCpr, chunk = lane % kCpr;
    const uint32_t dst_lane = (uint32_t)(chunk >> 3) * C::kChunkBytes;
    const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q;
    const __nv_bfloat16* kg = (const __nv_bfloat16*)p.k;
    const __nv_bfloat16* vg = (const __nv_bfloat16*)p.v;
    int32_t* const ktok_base = reinterpret_cast<int32_t*>(smem + C::kOffTok);
    int32_t* const qtok = reinterpret_cast<int32_t*>(smem + C::kOffQTok);
    uint32_t use = 0, gt = 0, it = 0;
    // A tile's barrier counts one arrival per producer thread, triggered by the hardware
    // when that thread's copies have landed (cp.async.mbarrier.arrive.noinc), so issuing
    // never waits for data.  The consumer publishes the data to the tensor core's proxy
    // (fence.proxy.async) after its wait.
    auto signal = [&](uint32_t mb) {
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(mb) : "memory");
    };
    auto wait_free = [&](uint32_t mb, uint32_t parity) {
      mbar_wait(mb, parity, gave_up, p.status);     // a failure sets *gave_up
    };
    // The rows of a tile are dealt to the three warps in groups of kRpi (group g to warp
    // g mod 3).  A warp takes four of its groups per pass (g, g+3, g+6, g+9): over a pass the
    // swizzle term of each of the four is the same in every pass (g advances by 12, and the
    // term only depends on g modulo 8 / kRpi), so it is prepared once per thread and the
    // destination of a copy is one addition away from the pass's base.
    constexpr int kGroups = kTile / kRpi;
    uint32_t sw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r7 = ((warp - 1 + 3 * k) * kRpi + sub) & 7;
      sw[k] = (uint32_t)(((chunk & 7) ^ r7) << 4) + (uint32_t)(3 * k * kRpi * 128);
    }
    auto gather = [&](const __nv_bfloat16* base, int64_t tok_stride, const int32_t* toks,
                      uint32_t dst_tile) {
      // token and token stride are both below 2^31: one 32 x 32 -> 64 bit multiply per row
      const uint32_t ts = (uint32_t)tok_stride * 2u;      // bytes
      const char* src0 = reinterpret_cast<const char*>(base + chunk * 8);
      const uint32_t dst0 = dst_tile + dst_lane + sub * 128;
      int grp = warp - 1;
      for (; grp + 9 < kGroups; grp += 12) {
        const int32_t* tk = toks + grp * kRpi + sub;
        const uint32_t d = dst0 + grp * (kRpi * 128);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const char* src = src0 + (uint64_t)(uint32_t)tk[3 * k * kRpi] * ts;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d + sw[k]), "l"(src)
                       : "memory");
        }
      }
      for (; grp < kGroups; grp += 3) {
        const int r = grp * kRpi + sub;
        const char* src = src0 + (uint64_t)(uint32_t)toks[r] * ts;
        const uint32_t dst = dst_tile + dst_lane + r * 128 + (((chunk & 7) ^ (r & 7)) << 4);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
      }
    };
    // Barrier over the three producer warps that also agrees on whether anyone in the CTA
    // has given up: every producer thread leaves the loops at the same point.
    auto group_sync_stop = [&]() {
      uint32_t any;
      asm volatile(
          "{\n\t.reg .pred p, q;\n\t"
          "setp.ne.u32 q, %1, 0;\n\t"
          "bar.red.or.pred p, 1, 96, q;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(any)
          : "r"((uint32_t)*gave_up)
          : "memory");
      return any != 0;
    };

    // ROPE: rows of a landed tile that this warp copied are turned in place.  A lane owns the
    // 16-byte piece `chunk` of its rows; the piece half a row further on holds the partner
    // dimensions (c <-> c + D/2).  Every lane reads both pieces, the warp meets, every lane
    // writes its own piece back: out = own * cos -/+ partner * sin (first / second half), in
    // fp32, rounded once to bf16 -- the arithmetic of the stand-alone rotation pass.
    auto rotate = [&](const int32_t* toks, uint32_t tile) {
      constexpr int kHalfC = kCpr / 2;
      const int pc = chunk < kHalfC ? chunk + kHalfC : chunk - kHalfC;
      const int fc = chunk < kHalfC ? chunk : chunk - kHalfC;
      const float sgn = chunk < kHalfC ? -1.f : 1.f;
      for (int grp = warp - 1; grp < kGroups; grp += 3) {
        const int r = grp * kRpi + sub;
        const uint32_t rb = tile + r * 128;
        const uint32_t a_own = rb + (uint32_t)(chunk >> 3) * C::kChunkBytes +
                               (uint32_t)(((chunk & 7) ^ (r & 7)) << 4);
        const uint32_t a_oth = rb + (uint32_t)(pc >> 3) * C::kChunkBytes +
                               (uint32_t)(((pc & 7) ^ (r & 7)) << 4);
        uint32_t own[4], oth[4];
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(own[0]), "=r"(own[1]), "=r"(own[2]), "=r"(own[3]) : "r"(a_own) : "memory");
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(oth[0]), "=r"(oth[1]), "=r"(oth[2]), "=r"(oth[3]) : "r"(a_oth) : "memory");
        const size_t at = (size_t)toks[r] * (D / 2) + 8 * fc;
        __syncwarp();
        uint32_t res[4];
#pragma unroll
        for (int hx = 0; hx < 2; ++hx) {           // four dimensions at a time: few live registers
          const float4 c4 = *reinterpret_cast<const float4*>(p.rope_cos + at + 4 * hx);
          const float4 s4 = *reinterpret_cast<const float4*>(p.rope_sin + at + 4 * hx);
          const float co[4] = {c4.x, c4.y, c4.z, c4.w}, si[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int w = 2 * hx + x;
            const float2 o = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&own[w]));
            const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&oth[w]));
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(
                fmaf(o.x, co[2 * x], sgn * (t.x * si[2 * x])),
                fmaf(o.y, co[2 * x + 1], sgn * (t.y * si[2 * x + 1])));
            res[w] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        }
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                     ::"r"(a_own), "r"(res[0]), "r"(res[1]), "r"(res[2]), "r"(res[3]) : "memory");
      }
    };
    auto commit_group = [&]() { asm volatile("cp.async.commit_group;" ::: "memory"); };

    bool live = true;
    for (int w_item = blockIdx.x; w_item < p.total_items && live; w_item += gridDim.x, ++it) {
      const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
      const int hk = bh % p.Hkv, b = bh / p.Hkv;
      const Geo g = make_geo(p, item, hk);
      const int32_t* perm = p.perm ? p.perm + (size_t)b * p.n : nullptr;
      const __nv_bfloat16* kb = kg + b * p.ks[0] + hk * p.ks[1];
      const __nv_bfloat16* vb = vg + b * p.ks[0] + hk * p.ks[1];
      auto key_tok = [&](int j, int r) {
        const int slot = actual_slot(p, g.kstart + j * kTile + r);
        return perm ? perm[slot] : slot;
      };
      auto q_tok = [&](int x) {        // x in 0..255: tile x/128, row x%128
        const int slot = min(g.q0[x >> 7] + (x & 127), p.n - 1);
        return perm ? perm[slot] : slot;
      };
      // tokens are fetched one tile ahead of their use
      int tk0 = key_tok(0, ptid), tk1 = ptid < 32 ? key_tok(0, ptid + 96) : 0;
      const int tq0 = q_tok(ptid), tq1 = q_tok(ptid + 96), tq2 = ptid < 64 ? q_tok(ptid + 192) : 0;
      for (int j = 0; j < g.T; ++j, ++gt) {
        // ---- K_j and the tokens of its keys
        if (use >= (uint32_t)C::kSlots)
          wait_free(bar(C::kBarSlotEmpty + use % C::kSlots), (use / C::kSlots - 1) & 1u);
        int32_t* ktok = ktok_base + (gt % C::kTok) * kTile;
        ktok[ptid] = tk0;
        if (ptid < 32) ktok[ptid + 96] = tk1;
        if (group_sync_stop()) { live = false; break; }
        if (ptid == 0) mbar_arrive(bar(C::kBarTokFull + gt % C::kTok));
        const uint32_t k_dst = sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes;
        const uint32_t k_bar = bar(C::kBarSlotFull + use % C::kSlots);
        gather(kb, p.ks[2], ktok, k_dst);
        if (ROPE) commit_group(); else signal(k_bar);
        ++use;
        if (j + 1 < g.T) {
          tk0 = key_tok(j + 1, ptid);
          if (ptid < 32) tk1 = key_tok(j + 1, ptid + 96);
        }
        if (j == 0) {
          // ---- Q of this item, once the products of the previous item no longer read it
          if (it >= (uint32_t)C::kQBufs)
            wait_free(bar(C::kBarQEmpty + it % C::kQBufs), (it / C::kQBufs - 1) & 1u);
          qtok[ptid] = tq0;
          qtok[ptid + 96] = tq1;
          if (ptid < 64) qtok[ptid + 192] = tq2;
          if (group_sync_stop()) { live = false; break; }
#pragma unroll
          for (int t = 0; t < 2; ++t)
            gather(qg + b * p.qs[0] + g.hq[t] * p.qs[1], p.qs[2], qtok + t * kTile,
                   sbase + C::kOffQ + (2 * (it % C::kQBufs) + t) * C::kTileBytes);
          if (ROPE) commit_group(); else signal(bar(C::kBarQFull + it % C::kQBufs));
        }
        // ---- V_j
        if (use >= (uint32_t)C::kSlots)
          wait_free(bar(C::kBarSlotEmpty + use % C::kSlots), (use / C::kSlots - 1) & 1u);
        if (group_sync_stop()) { live = false; break; }
        gather(vb, p.ks[2], ktok, sbase + C::kOffRing + (use % C::kSlots) * C::kTileBytes);
        signal(bar(C::kBarSlotFull + use % C::kSlots));
        ++use;
        if (ROPE) {
          // K_j (and Q at the start of an item) have landed once at most the V_j copies are
          // still under way; turn the rows, publish them to the tensor core's proxy, arrive
          commit_group();
          asm volatile("cp.async.wait_group 1;" ::: "memory");
          __syncwarp();
          rotate(ktok, k_dst);
          if (j == 0) {
            rotate(qtok, sbase + C::kOffQ + 2 * (it % C::kQBufs) * C::kTileBytes);
            rotate(qtok + kTile, sbase + C::kOffQ + (2 * (it % C::kQBufs) + 1) * C::kTileBytes);
          }
          fence_proxy_async();
          mbar_arrive(k_bar);
          if (j == 0) mbar_arrive(bar(C::kBarQFull + it % C::kQBufs));
        }
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // nothing in flight when the CTA leaves
  } else {
    // -------------------------------------------------------------- MMA issuer (warp 0)
    // One thread feeds the tensor core, so every instruction between two tcgen05.mma counts:
    // the descriptors are built from words prepared outside the loops and the K steps are
    // fully unrolled with immediate offsets.
    //
    // Scores are produced 64 keys at a time into the two halves of a tile's S columns, two
    // half-steps ahead of the softmax: while the softmax works on one half, the other half
    // already holds the next scores, so the softmax never waits for Q K^T and the tensor
    // core never waits for the softmax of the same tile.
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kTile, kHalf, false);
      constexpr uint32_t idesc_pv = instr_desc(kTile, D, true);
      // shared-memory descriptor words (128-byte swizzle, 1024 bytes between 8-row groups)
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t kLoK = (16u >> 4) << 16;                          // K-major operands
      constexpr uint32_t kLoV = ((uint32_t)C::kChunkBytes >> 4) << 16;     // V: next 64 columns
      const uint64_t q_first = desc64(((sbase + C::kOffQ) >> 4) | kLoK, kDescHi);
      uint64_t q_desc0 = q_first, q_desc1 = q_first + (C::kTileBytes >> 4);   // this item's Q tiles
      const uint32_t ring_lo = (sbase + C::kOffRing) >> 4;
      bool ok = true;
      uint32_t use = 0, it = 0;
      uint32_t pc00 = 0, pc01 = 0, pc10 = 0, pc11 = 0;   // p_ready waits so far, per [tile][half]
      auto slot_lo = [&](uint32_t u) { return ring_lo + (u % C::kSlots) * (C::kTileBytes >> 4); };
      auto slot_wait = [&](uint32_t u) {
        return mbar_wait(bar(C::kBarSlotFull + u % C::kSlots), (u / C::kSlots) & 1u, gave_up,
                         p.status);
      };
      // S(t, half b) = Q_t K^T over keys [64 b, 64 b + 64) of the K tile at k_lo
      auto issue_qk = [&](int t, int b, uint32_t k_lo) {
        const uint64_t qd = t ? q_desc1 : q_desc0;
        const uint64_t kd = desc64((k_lo + b * (kHalf * 128 >> 4)) | kLoK, kDescHi);
        const uint32_t d = tmem + t * 128 + b * kHalf;
        mma_ss_x4(d, qd, kd, idesc_qk, 0u);
        if (D == 128)   // columns 64..127 live one 16 KB block further on
          mma_ss_x4(d, qd + (C::kChunkBytes >> 4), kd + (C::kChunkBytes >> 4), idesc_qk, 1u);
        tc_commit(bar(C::kBarSFull + 2 * t + b));
      };
      // O_t += P(t, half b) V over the same 64 keys of the V tile at v_lo
      auto issue_pv = [&](int t, int b, uint32_t v_lo, uint32_t acc0) {
        const uint64_t vd = desc64((v_lo + b * (kHalf * 128 >> 4)) | kLoV, kDescHi);
        mma_ts_x4(tmem + C::kColO + t * D, tmem + t * 128 + b * kHalf, vd, idesc_pv, acc0);
        if (KB == 128)
          mma_ts_x4(tmem + C::kColO + t * D, tmem + t * 128 + 32, vd + 512, idesc_pv, 1u);
        // A commit holds the tensor pipe up for some 180 cycles, so none is spent where another
        // one already tells the same: with 128-key blocks the next scores of this tile follow
        // this product in the pipe, and their "S full" says that it is over as well.
        if (NB == 2) tc_commit(bar(C::kBarPvDone + t));
      };
      for (int w_item = blockIdx.x; w_item < p.total_items && ok; w_item += gridDim.x, ++it) {
        const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
        const Geo g = make_geo(p, item, bh % p.Hkv);
        const int H = NB * g.T;         // score blocks of this item
        // half-steps [first, last] that each query tile takes part in (a contiguous range);
        // everything per tile is kept in scalars so that nothing is indexed at run time
        int first0, first1, last0, last1;
        active_halves(p, g.q0[0], g.valid[0], g.kstart, H, kShift, &first0, &last0);
        active_halves(p, g.q0[1], g.valid[1], g.kstart, H, kShift, &first1, &last1);
        uint32_t started0 = 0, started1 = 0;
        // ring uses of this item: K_j = use + 2j, V_j = use + 2j + 1
        const uint32_t qb = it % C::kQBufs;
        q_desc0 = q_first + qb * (2 * C::kTileBytes >> 4);
        q_desc1 = q_desc0 + (C::kTileBytes >> 4);
        ok = mbar_wait(bar(C::kBarQFull + qb), (it / C::kQBufs) & 1u, gave_up, p.status);
        if (ok) ok = slot_wait(use);
        if (!ok) break;
        fence_proxy_async();
        tc_fence_after();
        {
          const uint32_t k0 = slot_lo(use);
          if (first0 <= 0 && last0 >= 0) issue_qk(0, 0, k0);
          if (first1 <= 0 && last1 >= 0) issue_qk(1, 0, k0);
          if (NB == 2) {
            if (first0 <= 1 && last0 >= 1) issue_qk(0, 1, k0);
            if (first1 <= 1 && last1 >= 1) issue_qk(1, 1, k0);
          }
        }
        tc_commit(bar(C::kBarSlotEmpty + use % C::kSlots));
        if (g.T == 1) tc_commit(bar(C::kBarQEmpty + qb));
        for (int j = 0; j < g.T && ok; ++j) {
          const uint32_t uv = use + 2 * j + 1, uk = use + 2 * j + 2;
          const bool more = j + 1 < g.T;
          // first touch of V_j and of K_{j+1}: both are needed within this step
          ok = slot_wait(uv);
          if (ok && more) ok = slot_wait(uk);
          if (!ok) break;
          fence_proxy_async();
          const uint32_t v_lo = slot_lo(uv), k_lo = slot_lo(uk);
          // one (tile, half) unit: P V of half-step h, then Q K^T of half-step h + 2
          auto unit = [&](auto tc, auto bc, int first, int last, uint32_t& started, uint32_t& pcnt) {
            constexpr int t = decltype(tc)::value, b = decltype(bc)::value;
            const int h = NB * j + b;
            if (h >= first && h <= last) {
              ok = mbar_wait(bar(C::kBarPReady + 2 * t + b), pcnt & 1u, gave_up, p.status);
              if (!ok) return;
              ++pcnt;
              tc_fence_after();
              issue_pv(t, b, v_lo, started);
              started = 1;
              if (h == last) tc_commit(bar(C::kBarODone + t));
            }
            if (more && h + NB >= first && h + NB <= last) issue_qk(t, b, k_lo);
          };
          using I0 = std::integral_constant<int, 0>;
          using I1 = std::integral_constant<int, 1>;
          unit(I0{}, I0{}, first0, last0, started0, pc00);
          if (ok) unit(I1{}, I0{}, first1, last1, started1, pc10);
          if (NB == 2) {
            if (ok) unit(I0{}, I1{}, first0, last0, started0, pc01);
            if (ok) unit(I1{}, I1{}, first1, last1, started1, pc11);
          }
          if (!ok) break;
          // the slots free when the products issued so far have finished
          tc_commit(bar(C::kBarSlotEmpty + uv % C::kSlots));
          if (more) tc_commit(bar(C::kBarSlotEmpty + uk % C::kSlots));
          if (j + 2 == g.T) tc_commit(bar(C::kBarQEmpty + qb));
        }
        use += 2 * g.T;
      }
    }
    __syncwarp();
  }
  } else {
    if (ROPE) asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    else asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    // ------------------------------------------------- softmax and epilogue
    const int t = (warp - 4) / 4;
    const int row = threadIdx.x - 128 - t * 128;       // 0..127 == TMEM lane
    const uint32_t lane_addr = (uint32_t)(row & ~31) << 16;
    const uint32_t s_addr = tmem + lane_addr + t * 128;
    const uint32_t o_addr = tmem + lane_addr + C::kColO + t * D;
    uint32_t s_cnt0 = 0, s_cnt1 = 0, o_cnt = 0, pv_cnt = 0, gt = 0, rows_cnt = 0;
    bool ok = true;

    // geometry and query token of an item; fetched one item ahead
    struct ItemCtx { int b, q0, hq, valid, kstart, T, first, last, q_tok; bool row_valid; };
    auto load_item = [&](int w_item) {
      ItemCtx c;
      const int item = w_item % p.items_per_kv, bh = w_item / p.items_per_kv;
      c.b = bh / p.Hkv;
      const Geo g = make_geo(p, item, bh % p.Hkv);
      c.q0 = t ? g.q0[1] : g.q0[0];
      c.hq = t ? g.hq[1] : g.hq[0];
      c.valid = t ? g.valid[1] : g.valid[0];
      c.kstart = g.kstart;
      c.T = g.T;
      active_halves(p, c.q0, c.valid, c.kstart, NB * c.T, kShift, &c.first, &c.last);
      const int qv = c.q0 + row;
      c.row_valid = c.valid && qv < p.n;
      c.q_tok = c.row_valid ? (p.perm ? p.perm[(size_t)c.b * p.n + qv] : qv) : 0;
      return c;
    };
    ItemCtx nxt{};
    if ((int)blockIdx.x < p.total_items) nxt = load_item(blockIdx.x);

    for (int w_item = blockIdx.x; w_item < p.total_items && ok; w_item += gridDim.x) {
      const ItemCtx cur = nxt;
      const int b = cur.b, q0 = cur.q0;
      const uint32_t gt0 = gt;
      gt += cur.T;
      if (!cur.valid) {
        if (w_item + (int)gridDim.x < p.total_items) nxt = load_item(w_item + gridDim.x);
        continue;
      }
      const int qv = q0 + row;
      const bool row_valid = cur.row_valid;
      const int q_tok = cur.q_tok;
      const int qcmp = (p.causal && !p.one_sided) ? q_tok : 0x7fffffff;
      if (COMBINE && !TMA && row_valid) {
        // the epilogue will read the other branch's row: start bringing it into L2 now
        const __nv_bfloat16* orow = (const __nv_bfloat16*)p.y_other + b * p.qs[0] +
                                    cur.hq * p.qs[1] + (int64_t)q_tok * p.qs[2];
#pragma unroll
        for (int x = 0; x < D * 2 / 128; ++x)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(orow + 64 * x));
      }
      float m = -INFINITY, l = 0.f;
      bool started = false;

      for (int h = cur.first; h <= cur.last; ++h) {
        const int kv = cur.kstart + h * kHalf;
        const int cls = tile_class(p, q0, kv, kHalf);
        const int hb = h & (NB - 1);
        const uint32_t tg = gt0 + (h >> (NB - 1));
        // the token list belongs to the whole 128-key tile: wait for it at its first half only
        if (hb == 0 || h == cur.first)
          ok = mbar_wait(bar(C::kBarTokFull + tg % C::kTok), (tg / C::kTok) & 1u, gave_up, p.status);
        if (ok)
          ok = mbar_wait(bar(C::kBarSFull + 2 * t + hb), (hb ? s_cnt1 : s_cnt0) & 1u, gave_up,
                         p.status);
        ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below are warp-collective
        if (!ok) break;
        s_cnt0 += 1 - hb;
        s_cnt1 += hb;
        tc_fence_after();

        const uint32_t sh_addr = s_addr + hb * kHalf;
        uint32_t sr[kHalf];
#pragma unroll
        for (int c = 0; c < kHalf / 32; ++c)
          tmem_ld32(sh_addr + 32 * c, reinterpret_cast<uint32_t(&)[32]>(sr[32 * c]));
        tmem_wait_ld();
        const int32_t* ktok = reinterpret_cast<const int32_t*>(smem + C::kOffTok) +
                              (tg % C::kTok) * kTile + hb * kHalf;
        if (cls == kCausalOnly) {
#pragma unroll
          for (int c = 0; c < kHalf; c += 4) {
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
          for (int c = 0; c < kHalf; c += 4) {
            const int4 kt = *reinterpret_cast<const int4*>(ktok + c);
            if ((uint32_t)(c - lo) > span || kt.x > qcmp) sr[c] = 0xff800000u;
            if ((uint32_t)(c + 1 - lo) > span || kt.y > qcmp) sr[c + 1] = 0xff800000u;
            if ((uint32_t)(c + 2 - lo) > span || kt.z > qcmp) sr[c + 2] = 0xff800000u;
            if ((uint32_t)(c + 3 - lo) > span || kt.w > qcmp) sr[c + 3] = 0xff800000u;
          }
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
#pragma unroll
        for (int c = 2; c < kHalf; c += 4) {
          mx0 = max3(mx0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
          if (c + 2 < kHalf)
            mx1 = max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
        }
        const float m_new = fmaxf(m, fmaxf(mx0, mx1));
        // Lazy rescaling: keep the old reference maximum while the new one is within 2^8.
        const bool grow = (m_new - m) * p.scale2 > 8.f || (m == -INFINITY && m_new > -INFINITY);
        if (!started) {
          m = m_new;
        } else if (__any_sync(0xffffffffu, grow)) {
          // O is still being accumulated by the previous P V: wait for it before touching O
          // (128-key blocks: these scores were issued behind that product, so it is over)
          if (NB == 2) {
            ok = mbar_wait(bar(C::kBarPvDone + t), (pv_cnt - 1) & 1u, gave_up, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
          }
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
        for (int c = 0; c < kHalf / 64; ++c) {
          uint32_t pk[32];          // 64 probabilities, two bf16 per word
#pragma unroll
          for (int x = 0; x < 32; ++x) {
            const float2 a = __ffma2_rn(make_float2(__uint_as_float(sr[64 * c + 2 * x]),
                                                    __uint_as_float(sr[64 * c + 2 * x + 1])),
                                        sc2, ng2);
            const float2 e = make_float2(exp2f(a.x), exp2f(a.y));
            lsum = __fadd2_rn(lsum, e);
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(e.x, e.y);
            pk[x] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          tmem_st32(sh_addr + 32 * c, pk);
        }
        l += lsum.x + lsum.y;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(C::kBarPReady + 2 * t + hb));
        ++pv_cnt;                           // the issuer answers every arrive with one P V
      }
      if (!ok) break;
      // fetch the next item's geometry and query token while the last products finish
      if (w_item + (int)gridDim.x < p.total_items) nxt = load_item(w_item + gridDim.x);

      ok = mbar_wait(bar(C::kBarODone + t), o_cnt & 1u, gave_up, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ++o_cnt;
      tc_fence_after();
      const float inv_l = 1.f / l;
      float g_this = 1.f, g_other = 0.f;
      const int hq = cur.hq;
      constexpr bool wc = COMBINE && TMA;   // with TMA tiles the gates are applied by warps 2 and 3
      if (COMBINE && !wc) {
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
        // Gated combine: this piece of the other branch's row (in L2 since the start of the
        // item) is requested before anything of the piece is stored, four loads in flight
        // together.  y may be the buffer the other rows sit in: a piece is read before the
        // same columns are written.
        uint4 oth[4];
        if (COMBINE && !wc && row_valid) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8)
            oth[x8] = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)p.y_other + off +
                                                      32 * c + 8 * x8);
        }
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
            if (COMBINE && !wc) {
              const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&oth[x8]);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                o[2 * x] = fmaf(g_other, __low2float(h2[x]), o[2 * x] * g_this);
                o[2 * x + 1] = fmaf(g_other, __high2float(h2[x]), o[2 * x + 1] * g_this);
              }
            }
            if (p.y && !(wc && p.y_branch)) {   // (wc: y is written by the combining warps)
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
      // rows of this tile are stored: the combining warps may take them (release at CTA scope),
      // once they have seen the arrival for the item before
      if (wc) {
        if (rows_cnt) ok = mbar_wait(bar(C::kBarRowsTaken + t), (rows_cnt - 1) & 1u, gave_up, p.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        mbar_arrive(bar(C::kBarRowsDone + t));
        ++rows_cnt;
      }
      // the next item's first P V overwrites O: order these reads before the arrive that
      // lets it start
      tc_fence_before();
    }
  }

  // ----------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------- host

// Score-block width.  Narrow windows skip more with 64-key blocks; from w = 256 on the
// 128-key block wins (half as many products, commits and softmax rounds per key).  The
// test hook sa_debug_set(SA_DEBUG_SCORE_BLOCK, 64 | 128) overrides the choice.
bool key_block_128(int w) {
  const int forced = debug_option(SA_DEBUG_SCORE_BLOCK);
  return forced ? forced == 128 : w > 128;
}

// sa_debug_set(SA_DEBUG_SWA_TILE_LOADS, 0) keeps the cp.async gather for the one-sided SWA
// branch too.
bool swa_tma_disabled() { return debug_option(SA_DEBUG_SWA_TILE_LOADS) == 0; }

bool tc_disabled() { return debug_option(SA_DEBUG_TENSOR_CORES) == 0; }

}  // namespace

bool tc_forward_supported(const FwdArgs& a, int dtype) {
  if (tc_disabled() || dtype != SA_BF16 || (a.d != 128 && a.d != 64)) return false;
  if (a.n < 1 || (int64_t)a.B * a.Hq * ((a.n + kTile - 1) / kTile) > 0x3fffffff) return false;
  if (a.qs[2] >= (1ll << 30) || a.ks[2] >= (1ll << 30)) return false;   // 32-bit row strides
  return true;
}

cudaError_t launch_fwd_tc(const FwdArgs& a, cudaStream_t st) {
  TcParams p{};
  p.q = a.q; p.k = a.k; p.v = a.v;
  p.perm = a.swa ? nullptr : a.perm;
  p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin;
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
  for (int i = 0; i < 3; ++i) { p.qs[i] = a.qs[i]; p.ks[i] = a.ks[i]; }
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
  const bool wide = key_block_128(a.w);
  // whole-tile TMA loads for the one-sided SWA branch (any strides the maps can express;
  // otherwise the gather serves this branch too)
  CUtensorMap tm_q{}, tm_k{}, tm_v{};
  const bool rows_have_a_home =
      !(a.gate_logits && a.y_other) || (a.y_branch ? a.y_branch != a.y_other : a.y != a.y_other);
  if (a.swa && mg.one_sided && !swa_tma_disabled() && !a.rope_cos &&   // TMA tiles cannot be turned
      rows_have_a_home) {
    if (aligned16(a.q) && aligned16(a.k) && aligned16(a.v) &&
        make_map_bhnd(&tm_q, a.q, a.B, a.Hq, a.n, a.d, a.qs) &&
        make_map_bhnd(&tm_k, a.k, a.B, a.Hkv, a.n, a.d, a.ks) &&
        make_map_bhnd(&tm_v, a.v, a.B, a.Hkv, a.n, a.d, a.ks))
      p.use_tma = 1;
  }
  auto go = [&](auto kernel, int smem) {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    kernel<<<grid, kThreads, smem, st>>>(p, tm_q, tm_k, tm_v);
    return cudaSuccess;
  };
  const bool tma = p.use_tma != 0;
  const bool combine = a.gate_logits && a.y_other;
  // (checked below: the TMA variant combines with its idle warps, which needs this branch's rows
  // to have a home that is not the buffer the other branch's rows sit in)
  if (a.gate_logits && !a.y_other) return cudaErrorInvalidValue;   // gates only with the other rows
  // instantiation by (head dimension, score-block width, tile loads, rotation, combine)
  auto pick = [&](auto d_c, auto kb_c) {
    constexpr int DD = decltype(d_c)::value, KK = decltype(kb_c)::value;
    if (a.rope_cos)
      return combine ? go(fwd_tc_kernel<DD, KK, false, true, true>, Cfg<DD>::kBytes)
                     : go(fwd_tc_kernel<DD, KK, false, true, false>, Cfg<DD>::kBytes);
    if (tma)
      return combine ? go(fwd_tc_kernel<DD, KK, true, false, true>, Cfg<DD>::kBytes)
                     : go(fwd_tc_kernel<DD, KK, true, false, false>, Cfg<DD>::kBytes);
    return combine ? go(fwd_tc_kernel<DD, KK, false, false, true>, Cfg<DD>::kBytes)
                   : go(fwd_tc_kernel<DD, KK, false, false, false>, Cfg<DD>::kBytes);
  };
  using I64 = std::integral_constant<int, 64>;
  using I128 = std::integral_constant<int, 128>;
  if (a.d == 128) e = wide ? pick(I128{}, I128{}) : pick(I128{}, I64{});
  else e = wide ? pick(I64{}, I128{}) : pick(I64{}, I64{});
  if (e != cudaSuccess) return e;
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa
