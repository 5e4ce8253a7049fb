// Backward pass on the 5th-generation tensor cores, bf16, d = 64 or 128.
//
// Formulas (derivative of Eq. 1 with the permutation held constant; per branch x, with
// dO = g_x dY and Delta_i = g_x sum_c dY[i,c] Y_x[i,c] prepared by the delta kernel):
//   P_ij = exp(scale q_i.k_j - lse_i),  dP_ij = dY_i . v_j,
//   dS_ij = scale P_ij (g_x dP_ij - Delta_i),
//   dQ_i = sum_j dS_ij k_j,   dK_j = sum_i dS_ij q_i,   dV_j = sum_i g_x P_ij dY_i.
//
// Two launches per branch, neither of which needs an atomic, so results are run-to-run
// identical:
//   rows = queries: a CTA owns 128 query slots of one head, walks the K/V tiles of its
//                   band, and accumulates dQ;
//   rows = keys:    a CTA owns 128 key slots of one KV head, walks the query tiles that can
//                   see them for every query head of the group, and accumulates dK and dV.
// Either way one step is: S = R1 C1^T and dP = R2 C2^T into tensor memory (rows: Q, dY or
// K, V; columns: K, V or Q, dY), one thread per row turns them into P and dS (bf16, written
// back over S and dP), then dS (and P) multiply the column tiles into the accumulators.
// Rows of every operand are gathered through perm with cp.async into swizzled shared
// memory, as in the forward kernel; finished rows are scattered to their original places.
//
// The column tile is 128 or 64 wide (template KC).  64 halves the band-edge waste of narrow
// windows and, where scores and accumulators then fit in 256 tensor-memory columns, lets two
// CTAs share an SM so that one CTA's loads and epilogue hide behind the other's products.
//
// With NBUF = 2 (64-wide column tiles only) the scores of two consecutive column tiles live
// side by side in tensor memory: the products of tile i+1 run while the row threads work on
// tile i, and two warpgroups of row threads split a tile's 64 columns.
//
// Warp roles: warp 0 MMA issuer and TMEM allocator, warps 1-3 gather producers, then one
// (NBUF = 1) or two (NBUF = 2) warpgroups with one thread per row.  Every mbarrier wait is
// bounded.
#include <type_traits>

#include "sa_bwd_tc.cuh"
#include "sa_gemm_common.cuh"
#include "sa_tc_common.cuh"

namespace sa {
namespace {

constexpr int kTile = 128;
constexpr int kProducers = 96;

struct BwdTcParams {
  const void *q, *k, *v, *dy;
  const int32_t* perm;        // null for the SWA branch
  const float* lse;           // [B,Hq,n] of this branch
  const float* delta;         // [B,Hq,n] of this branch (gate included)
  const float* gate_logit;    // null, or the [Hq] logits of this branch
  void *dq, *dk, *dv;
  int accumulate;             // add to what the outputs already hold
  int* status;
  const int* abort_flag;
  int B, Hq, Hkv, G, n, w, h;
  int causal, linear, one_sided, full_range;
  int n_tiles;
  float scale, scale2;
  int64_t qs[3], ks[3];
};

// Columns (virtual slots) a row tile starting at slot r0 has to meet: [cstart, cend].
// rows_are_keys selects the transposed window of the one-sided rule.
__device__ __forceinline__ void column_range(const BwdTcParams& p, int r0, bool rows_are_keys,
                                             int kc, int* cstart, int* T) {
  const int rl = min(r0 + kTile - 1, p.n - 1);
  int lo, hi;
  if (p.full_range) { lo = 0; hi = p.n - 1; }
  else if (p.one_sided) {
    if (rows_are_keys) { lo = r0; hi = min(rl + p.w - 1, p.n - 1); }
    else { lo = max(r0 - (p.w - 1), 0); hi = rl; }
  } else if (p.linear) { lo = max(r0 - p.h, 0); hi = min(rl + p.h, p.n - 1); }
  else { lo = r0 - p.h; hi = rl + p.h; }
  *cstart = lo;
  *T = (hi - lo + kc) / kc;
}

__device__ __forceinline__ int actual_slot(const BwdTcParams& p, int v) {
  if (p.full_range || p.linear || p.one_sided) return min(max(v, 0), p.n - 1);
  v %= p.n;
  return v < 0 ? v + p.n : v;
}

// RW: warpgroups of row threads.  Two split a column tile's 32-column pieces between them: with
// two score buffers (products of the next tile overlap the row work) or, for 128-wide tiles,
// with one buffer, where they halve the time the tensor core waits for the row threads.
template <int D, int KC, int MODE, int NBUF, int RW>
struct BCfg {
  static_assert(NBUF == 1 || KC == 64, "two score buffers need 64-wide column tiles");
  static_assert(RW == 1 || RW == 2, "one or two warpgroups of row threads");
  static constexpr int kRowWgs = RW;                            // warpgroups of row threads
  static constexpr int kThreads = 128 + 128 * kRowWgs;
  static constexpr int kTileBytes = kTile * D * 2;              // a row-operand tile
  static constexpr int kChunkBytes = kTile * 128;               // its 64-column blocks
  static constexpr int kColBytes = KC * D * 2;                  // a column tile
  static constexpr int kColChunkBytes = KC * 128;
  static constexpr int kStages = NBUF == 2 ? 4 : 2;
  static constexpr int kOffR = 0;                               // two row-operand tiles
  static constexpr int kOffC = 2 * kTileBytes;                  // kStages x two column tiles
  static constexpr int kOffRowTok = kOffC + kStages * 2 * kColBytes;
  static constexpr int kOffColTok = kOffRowTok + kTile * 4;     // kStages x 128 ints
  static constexpr int kOffColVec = kOffColTok + kStages * kTile * 4;  // kStages x 2 x 128 floats
  static constexpr int kOffBar = kOffColVec + kStages * 2 * kTile * 4;
  static constexpr int kBarRFull = 0, kBarCFull = 1, kBarCEmpty = kBarCFull + kStages,
                       kBarTokFull = kBarCEmpty + kStages, kBarSFull = kBarTokFull + kStages,
                       kBarPReady = kBarSFull + NBUF, kBarODone = kBarPReady + NBUF,
                       kNumBars = kBarODone + 1;
  static constexpr int kOffMisc = kOffBar + kNumBars * 8;
  static constexpr int kBytes = kOffMisc + 16;
  // tensor memory columns: S and dS (NBUF buffers of KC) at 0, then dP and P, then the
  // accumulators
  static constexpr uint32_t kColS = 0, kColP = KC * NBUF, kColAcc = 2 * KC * NBUF;
  static constexpr uint32_t kColsUsed = 2 * KC * NBUF + (MODE == 1 ? 2 : 1) * D;
  static constexpr uint32_t kTmemCols = kColsUsed <= 256 ? 256 : 512;
  static constexpr int kCtasPerSm = (kTmemCols == 256 && kBytes <= 110 * 1024) ? 2 : 1;
  static_assert(kBytes <= 232448, "shared memory");
};

// MODE 0: rows are queries (dQ).  MODE 1: rows are keys (dK, dV).
// TMA: the instantiation for the one-sided SWA branch, whose rows are consecutive tokens: one
// warp loads whole tiles with cp.async.bulk.tensor (every CTA its own) instead of three warps
// gathering rows 16 bytes at a time, which is bound by the load/store unit.
template <int D, int KC, int MODE, int NBUF, int RW, bool TMA>
__global__ void __launch_bounds__(BCfg<D, KC, MODE, NBUF, RW>::kThreads,
                                  BCfg<D, KC, MODE, NBUF, RW>::kCtasPerSm)
bwd_tc_kernel(const __grid_constant__ BwdTcParams p, const __grid_constant__ CUtensorMap tm_q,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
              const __grid_constant__ CUtensorMap tm_dy) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using C = BCfg<D, KC, MODE, NBUF, RW>;
  constexpr uint32_t kTmemCols = C::kTmemCols;
  constexpr bool kKeys = MODE == 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {
    if (threadIdx.x == 0) atomicCAS(p.status, SA_OK, SA_ERR_CUDA);
    return;
  }
  const uint32_t bar0 = sbase + C::kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* gave_up = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);

  // work item: (batch, head of the row operand, row tile)
  const int H = kKeys ? p.Hkv : p.Hq;
  const int tile = blockIdx.x % p.n_tiles, bh = blockIdx.x / p.n_tiles;
  const int hr = bh % H, b = bh / H;
  const int hk = kKeys ? hr : hr / p.G;
  const int r0 = tile * kTile;
  int cstart, T;
  column_range(p, r0, kKeys, KC, &cstart, &T);
  const int iters = kKeys ? T * p.G : T;      // column tiles (times query heads of the group)
  const int32_t* perm = p.perm ? p.perm + (size_t)b * p.n : nullptr;

  if (threadIdx.x == 0) {
    *gave_up = 0;
    note_skip(reinterpret_cast<volatile int*>(smem + C::kOffMisc + 8), p.status, p.abort_flag);
    for (int i = 0; i < C::kNumBars; ++i)
      mbar_init(bar(i), (i >= C::kBarPReady && i < C::kBarODone) ? kTile * C::kRowWgs
                        : (i == C::kBarRFull || (i >= C::kBarCFull && i < C::kBarCEmpty))
                            ? (TMA ? 32 : kProducers) : 1);
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

  if (warp >= 1 && warp < 4 && TMA) {
    // ------------------------------------------------- tile loads by TMA (warp 1 alone)
    // Rows and columns are consecutive tokens (no permutation, window by slots only), so a tile
    // is D / 64 boxes of KC tokens x 64 columns per operand; tokens outside the sequence read
    // zeros and are masked by the slot window.  Lane 0 posts the byte counts and the loads;
    // for rows = keys the 32 lanes also fetch the per-query lse and delta of the columns.
    // The token lists are not written: the one-sided rule does not look at them.
    if (warp == 1) {
      auto signal = [&](uint32_t mb) {
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(mb) : "memory");
      };
      auto load_rows = [&](const CUtensorMap* tm, uint32_t dst, int tok, int head, int rows,
                           uint32_t mb) {
        for (int r = 0; r < rows; r += KC)
#pragma unroll
          for (int c = 0; c < D / 64; ++c)
            tma_load_4d(dst + c * (rows * 128) + r * 128, tm, 64 * c, tok + r, head, b, mb);
      };
      if (lane == 0) {
        mbar_expect_tx(bar(C::kBarRFull), 2 * C::kTileBytes);   // counts as this lane's arrival
        load_rows(kKeys ? &tm_k : &tm_q, sbase + C::kOffR, r0, hr, kTile, bar(C::kBarRFull));
        load_rows(kKeys ? &tm_v : &tm_dy, sbase + C::kOffR + C::kTileBytes, r0, hr, kTile,
                  bar(C::kBarRFull));
      } else {
        mbar_arrive(bar(C::kBarRFull));
      }
      bool live = true;
      int issued = 0;
      for (int it = 0; it < iters && live; ++it) {
        const int s = it % C::kStages;
        const int j = kKeys ? it % T : it, gi = kKeys ? it / T : 0;
        const int hq = kKeys ? hk * p.G + gi : hr;
        if (it >= C::kStages)
          live = mbar_wait(bar(C::kBarCEmpty + s), (it / C::kStages - 1) & 1u, gave_up, p.status);
        live = __all_sync(0xffffffffu, live);
        if (!live) break;
        issued = it + 1;
        const uint32_t colvec = sbase + C::kOffColVec + s * 2 * kTile * 4;
        const uint32_t c1 = sbase + C::kOffC + s * 2 * C::kColBytes, c2 = c1 + C::kColBytes;
        const uint32_t mb = bar(C::kBarCFull + s);
        if (lane == 0) mbar_arrive(bar(C::kBarTokFull + s));
        if (kKeys) {
          const float* lse_h = p.lse + ((size_t)b * p.Hq + hq) * p.n;
          const float* del_h = p.delta + ((size_t)b * p.Hq + hq) * p.n;
          // (lanes 1-31: lane 0 arrives by posting the byte count, which does not wait for
          // copies of its own)
          for (int x = lane - 1; x < KC && lane > 0; x += 31) {
            const int t0 = actual_slot(p, cstart + j * KC + x);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * x), "l"(lse_h + t0) : "memory");
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * (kTile + x)), "l"(del_h + t0) : "memory");
          }
        }
        if (lane == 0) {
          mbar_expect_tx(mb, 2 * C::kColBytes);                 // this lane's arrival
          load_rows(kKeys ? &tm_q : &tm_k, c1, cstart + j * KC, kKeys ? hq : hk, KC, mb);
          load_rows(kKeys ? &tm_dy : &tm_v, c2, cstart + j * KC, kKeys ? hq : hk, KC, mb);
        } else {
          signal(mb);                                           // after this lane's small copies
        }
      }
      asm volatile("cp.async.wait_all;" ::: "memory");
      // loads that were started but never consumed (only after a failed wait) must land before
      // the shared memory goes away: wait for them, again with a limit
      if (lane == 0 && (!live || *gave_up)) {
        for (int tries = 0; tries < 100000; ++tries) {
          if (mbar_try(bar(C::kBarRFull), 0u)) break;
          __nanosleep(100);
        }
        for (int u = issued > C::kStages ? issued - C::kStages : 0; u < issued; ++u)
          for (int tries = 0; tries < 100000; ++tries) {
            if (mbar_try(bar(C::kBarCFull + u % C::kStages), (u / C::kStages) & 1u)) break;
            __nanosleep(100);
          }
      }
    }
  } else if (warp >= 1 && warp < 4) {
    // ---------------------------------------------------- gather producers (warps 1-3)
    constexpr int kCpr = D / 8;            // 16-byte pieces per row
    constexpr int kRpi = 32 / kCpr;        // rows per warp instruction
    const int ptid = threadIdx.x - 32;     // 0..95
    const int sub = lane / kCpr, chunk = lane % kCpr;
    const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q;
    const __nv_bfloat16* kg = (const __nv_bfloat16*)p.k;
    const __nv_bfloat16* vg = (const __nv_bfloat16*)p.v;
    const __nv_bfloat16* dyg = (const __nv_bfloat16*)p.dy;
    int32_t* const rowtok = reinterpret_cast<int32_t*>(smem + C::kOffRowTok);
    auto signal = [&](uint32_t mb) {
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(mb) : "memory");
    };
    // rows x D elements into a tile whose 64-column blocks are rows x 128 bytes each
    auto gather = [&](const __nv_bfloat16* base, int64_t tok_stride, const int32_t* toks,
                      uint32_t dst_tile, int rows) {
#pragma unroll 4
      for (int grp = warp - 1; grp < rows / kRpi; grp += 3) {
        const int r = grp * kRpi + sub;
        const __nv_bfloat16* src = base + (int64_t)toks[r] * tok_stride + chunk * 8;
        const uint32_t dst = dst_tile + (uint32_t)(chunk >> 3) * (rows * 128) + r * 128 +
                             (((chunk & 7) ^ (r & 7)) << 4);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
      }
    };
    // Barrier over the three producer warps that also agrees on whether anyone in the CTA
    // has given up, so that every producer thread leaves at the same point.
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
    auto tok_of = [&](int slot) { return perm ? perm[slot] : slot; };

    // row operands
    rowtok[ptid] = tok_of(min(r0 + ptid, p.n - 1));
    if (ptid < 32) rowtok[ptid + 96] = tok_of(min(r0 + ptid + 96, p.n - 1));
    bool live = !group_sync_stop();
    if (live) {
      if (kKeys) {
        gather(kg + b * p.ks[0] + hr * p.ks[1], p.ks[2], rowtok, sbase + C::kOffR, kTile);
        gather(vg + b * p.ks[0] + hr * p.ks[1], p.ks[2], rowtok, sbase + C::kOffR + C::kTileBytes, kTile);
      } else {
        gather(qg + b * p.qs[0] + hr * p.qs[1], p.qs[2], rowtok, sbase + C::kOffR, kTile);
        gather(dyg + b * p.qs[0] + hr * p.qs[1], p.qs[2], rowtok, sbase + C::kOffR + C::kTileBytes, kTile);
      }
      signal(bar(C::kBarRFull));
    }
    // The tokens of a column tile come from global memory (perm); they are fetched one tile
    // ahead of their use so that this latency is not paid inside every step.
    auto col_tok = [&](int it, int x) {
      const int j = kKeys ? it % T : it;
      return tok_of(actual_slot(p, cstart + j * KC + x));
    };
    int nt0 = 0, nt1 = 0;
    if (live && iters > 0) {
      if (ptid < KC) nt0 = col_tok(0, ptid);
      if (ptid + 96 < KC) nt1 = col_tok(0, ptid + 96);
    }
    for (int it = 0; it < iters && live; ++it) {
      const int s = it % C::kStages;
      const int gi = kKeys ? it / T : 0;
      const int hq = kKeys ? hk * p.G + gi : hr;
      const int t0 = nt0, t1 = nt1;
      if (it + 1 < iters) {
        if (ptid < KC) nt0 = col_tok(it + 1, ptid);
        if (ptid + 96 < KC) nt1 = col_tok(it + 1, ptid + 96);
      }
      if (it >= C::kStages)
        mbar_wait(bar(C::kBarCEmpty + s), (it / C::kStages - 1) & 1u, gave_up, p.status);
      int32_t* coltok = reinterpret_cast<int32_t*>(smem + C::kOffColTok) + s * kTile;
      const uint32_t colvec = sbase + C::kOffColVec + s * 2 * kTile * 4;
      if (ptid < KC) coltok[ptid] = t0;
      if (ptid + 96 < KC) coltok[ptid + 96] = t1;
      if (group_sync_stop()) { live = false; break; }
      if (ptid == 0) mbar_arrive(bar(C::kBarTokFull + s));
      const uint32_t c1 = sbase + C::kOffC + s * 2 * C::kColBytes, c2 = c1 + C::kColBytes;
      if (kKeys) {
        // per-query vectors of this head travel with the tile
        const float* lse_h = p.lse + ((size_t)b * p.Hq + hq) * p.n;
        const float* del_h = p.delta + ((size_t)b * p.Hq + hq) * p.n;
        if (ptid < KC) {
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * ptid), "l"(lse_h + t0) : "memory");
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * (kTile + ptid)), "l"(del_h + t0) : "memory");
        }
        if (ptid + 96 < KC) {
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * (ptid + 96)), "l"(lse_h + t1) : "memory");
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(colvec + 4 * (kTile + ptid + 96)), "l"(del_h + t1) : "memory");
        }
        gather(qg + b * p.qs[0] + hq * p.qs[1], p.qs[2], coltok, c1, KC);
        gather(dyg + b * p.qs[0] + hq * p.qs[1], p.qs[2], coltok, c2, KC);
      } else {
        gather(kg + b * p.ks[0] + hk * p.ks[1], p.ks[2], coltok, c1, KC);
        gather(vg + b * p.ks[0] + hk * p.ks[1], p.ks[2], coltok, c2, KC);
      }
      signal(bar(C::kBarCFull + s));
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // nothing in flight when the CTA leaves
  } else if (warp == 0) {
    // -------------------------------------------------------------- MMA issuer (warp 0)
    if (lane == 0) {
      constexpr uint32_t idesc_s = instr_desc(kTile, KC, false);
      constexpr uint32_t idesc_acc = instr_desc(kTile, D, true);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t kLoK = (16u >> 4) << 16;                        // K-major operands
      constexpr uint32_t kLoMN = ((uint32_t)C::kColChunkBytes >> 4) << 16;  // column tile as [k][n]
      constexpr uint32_t kBlockR = C::kChunkBytes >> 4;     // next 64 columns of a row tile
      constexpr uint32_t kBlockC = C::kColChunkBytes >> 4;  // next 64 columns of a column tile
      const uint64_t r1 = desc64(((sbase + C::kOffR) >> 4) | kLoK, kDescHi);
      const uint64_t r2 = desc64(((sbase + C::kOffR + C::kTileBytes) >> 4) | kLoK, kDescHi);
      // X (128 x 128, fp32, tensor memory column col) = A B^T, both tiles K-major, K = D
      auto product = [&](uint32_t col, uint64_t a, uint32_t b_addr) {
        const uint64_t bd = desc64((b_addr >> 4) | kLoK, kDescHi);
        mma_ss_x4(tmem + col, a, bd, idesc_s, 0u);
        if (D == 128) mma_ss_x4(tmem + col, a + kBlockR, bd + kBlockC, idesc_s, 1u);
      };
      // acc (128 x D, tensor memory column col) += X (bf16 pairs at column xcol) * tile
      auto accumulate = [&](uint32_t col, uint32_t xcol, uint32_t b_addr, uint32_t acc0) {
        const uint64_t bd = desc64((b_addr >> 4) | kLoMN, kDescHi);
        mma_ts_x4(tmem + col, tmem + xcol, bd, idesc_acc, acc0);
        if (KC == 128) mma_ts_x4(tmem + col, tmem + xcol + 32, bd + 512, idesc_acc, 1u);
      };
      // scores of column tile `it` into buffer it % NBUF
      auto scores = [&](int it) {
        const int s = it % C::kStages;
        const uint32_t c1 = sbase + C::kOffC + s * 2 * C::kColBytes, c2 = c1 + C::kColBytes;
        if (!mbar_wait(bar(C::kBarCFull + s), (it / C::kStages) & 1u, gave_up, p.status))
          return false;
        fence_proxy_async();
        tc_fence_after();
        const uint32_t buf = (it % NBUF) * KC;
        product(C::kColS + buf, r1, c1);
        product(C::kColP + buf, r2, c2);
        tc_commit(bar(C::kBarSFull + it % NBUF));
        return true;
      };
      bool ok = mbar_wait(bar(C::kBarRFull), 0, gave_up, p.status);
      if (ok && NBUF == 2) ok = scores(0);
      for (int it = 0; it < iters && ok; ++it) {
        const int s = it % C::kStages;
        const uint32_t c1 = sbase + C::kOffC + s * 2 * C::kColBytes, c2 = c1 + C::kColBytes;
        // NBUF = 2: the next tile's scores go ahead of this tile's accumulation
        if (NBUF == 2) { if (it + 1 < iters) ok = scores(it + 1); }
        else ok = scores(it);
        if (!ok) break;
        ok = mbar_wait(bar(C::kBarPReady + it % NBUF), (it / NBUF) & 1u, gave_up, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t buf = (it % NBUF) * KC;
        if (kKeys) {
          accumulate(C::kColAcc, C::kColP + buf, c2, it > 0);        // dV += (g P)^T dY
          accumulate(C::kColAcc + D, C::kColS + buf, c1, it > 0);    // dK += dS^T Q
        } else {
          accumulate(C::kColAcc, C::kColS + buf, c1, it > 0);        // dQ += dS K
        }
        tc_commit(bar(C::kBarCEmpty + s));
      }
      if (ok) tc_commit(bar(C::kBarODone));
    }
    __syncwarp();
  } else {
    // ------------------------------------------------- row threads (from warp 4 on)
    const int wg = (warp - 4) >> 2;                     // which warpgroup of row threads
    const int row = (threadIdx.x - 128) & 127;          // 0..127 == TMEM lane
    const uint32_t trow = tmem + ((uint32_t)(row & ~31) << 16);
    const int rslot = r0 + row;
    const bool row_valid = rslot < p.n;
    const int rtok = perm ? perm[min(rslot, p.n - 1)] : min(rslot, p.n - 1);
    const bool tok_rule = p.causal && !p.one_sided;     // token order decides, not slots
    // rows = queries: mask key tokens above the query's; rows = keys: query tokens below
    const int cmp = tok_rule ? rtok : (kKeys ? (int)0x80000000 : 0x7fffffff);
    // exp2(s * scale2 - lse2 + log2(scale)) is P * scale at once: dS needs no further multiply
    const float l2scale = __log2f(p.scale), inv_scale = 1.f / p.scale;
    float lse2_r = 0.f, delta_r = 0.f, g = 1.f;
    if (!kKeys) {
      const size_t o = ((size_t)b * p.Hq + hr) * p.n + rtok;
      lse2_r = p.lse[o] * kLog2e - l2scale;
      delta_r = p.delta[o];
      if (p.gate_logit) g = 1.f / (1.f + __expf(-p.gate_logit[hr]));
    }
    // Two warpgroups share a tile: the bf16 results of one overwrite score columns the other
    // reads, so every row thread loads before any stores.  The barrier also agrees on whether
    // to stop, so that all of them leave the loop together.
    auto rows_sync_stop = [&](bool stop) {
      uint32_t any;
      asm volatile(
          "{\n\t.reg .pred p, q;\n\t"
          "setp.ne.u32 q, %1, 0;\n\t"
          "bar.red.or.pred p, 2, 256, q;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(any)
          : "r"((uint32_t)stop)
          : "memory");
      return any != 0;
    };
    bool ok = true;
    for (int it = 0; it < iters; ++it) {
      const int s = it % C::kStages;
      const uint32_t buf = (it % NBUF) * KC;
      const int j = kKeys ? it % T : it;
      if (kKeys && p.gate_logit) g = 1.f / (1.f + __expf(-p.gate_logit[hk * p.G + it / T]));
      ok = mbar_wait(bar(C::kBarTokFull + s), (it / C::kStages) & 1u, gave_up, p.status);
      if (ok) ok = mbar_wait(bar(C::kBarSFull + it % NBUF), (it / NBUF) & 1u, gave_up, p.status);
      ok = __all_sync(0xffffffffu, ok);   // the tensor-memory accesses below are warp-collective
      if (C::kRowWgs == 1 && !ok) break;
      if (ok) tc_fence_after();
      // visible columns of this row: one interval [lo, lo + span], cut by the token order
      const int cb = cstart + j * KC;
      const bool clamp = p.linear || p.full_range || p.one_sided;
      int lo, hi;
      if (p.one_sided) {
        if (kKeys) { lo = rslot - cb; hi = p.full_range ? p.n - 1 - cb : rslot + (p.w - 1) - cb; }
        else { lo = p.full_range ? -cb : rslot - (p.w - 1) - cb; hi = rslot - cb; }
      } else if (p.full_range && !p.linear) { lo = -cb; hi = p.n - 1 - cb; }
      else { lo = rslot - p.h - cb; hi = rslot + p.h - cb; }
      // Every row of the tile sees every column of this tile (up to the token order) when the
      // last row's interval starts at or before column 0, the first row's ends at or after the
      // last column and no clamp cuts in: then the per-element interval test is left out.
      // (The interval moves with the row's slot, one column per row.)
      const bool interior = !p.full_range && lo + (kTile - 1 - row) <= 0 && hi - row >= KC - 1 &&
                            (!clamp || (cb >= 0 && cb + KC <= p.n)) && r0 + kTile - 1 < p.n;
      if (clamp) {
        lo = max(lo, -cb);
        hi = min(hi, p.n - 1 - cb);
      }
      if (hi < lo) { lo = 1 << 30; hi = lo; }
      const uint32_t span = (uint32_t)(hi - lo);
      const int32_t* coltok = reinterpret_cast<const int32_t*>(smem + C::kOffColTok) + s * kTile;
      const float* colvec = reinterpret_cast<const float*>(smem + C::kOffColVec) + s * 2 * kTile;
#pragma unroll 1
      for (int c = wg; c < KC / 32; c += C::kRowWgs) {
        uint32_t sv[32], dv[32];
        if (ok) {
          tmem_ld32(trow + C::kColS + buf + 32 * c, sv);
          tmem_ld32(trow + C::kColP + buf + 32 * c, dv);
          tmem_wait_ld();
        }
        if (C::kRowWgs == 2 && rows_sync_stop(!ok)) { ok = false; break; }
        uint32_t ds_pk[16], p_pk[16];
        auto chunk = [&](auto inter_c) {
        constexpr bool kInter = decltype(inter_c)::value;
        // TMA tiles are the one-sided local branch: slots decide, the token lists are not even
        // written, and their loads would only take shared-memory bandwidth from the products
        constexpr bool kTok = !TMA;
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
          const int col = 32 * c + x;
          int4 ct = make_int4(0, 0, 0, 0);
          if (kTok) ct = *reinterpret_cast<const int4*>(coltok + col);
          float4 l4 = make_float4(lse2_r, lse2_r, lse2_r, lse2_r);
          float4 d4 = make_float4(delta_r, delta_r, delta_r, delta_r);
          if (kKeys) {
            l4 = *reinterpret_cast<const float4*>(colvec + col);
            l4.x = fmaf(l4.x, kLog2e, -l2scale); l4.y = fmaf(l4.y, kLog2e, -l2scale);
            l4.z = fmaf(l4.z, kLog2e, -l2scale); l4.w = fmaf(l4.w, kLog2e, -l2scale);
            d4 = *reinterpret_cast<const float4*>(colvec + kTile + col);
          }
          const int ctk[4] = {ct.x, ct.y, ct.z, ct.w};
          const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dl[4] = {d4.x, d4.y, d4.z, d4.w};
          float pv[4], dsv[4];
          const float gp = g * inv_scale;
          // two elements per instruction where the operation has a packed form
          const float2 sc2 = make_float2(p.scale2, p.scale2), g2 = make_float2(g, g);
#pragma unroll
          for (int y = 0; y < 4; y += 2) {
            const bool vis0 = (kInter || (uint32_t)(col + y - lo) <= span) &&
                              (!kTok || (kKeys ? ctk[y] >= cmp : ctk[y] <= cmp));
            const bool vis1 = (kInter || (uint32_t)(col + y + 1 - lo) <= span) &&
                              (!kTok || (kKeys ? ctk[y + 1] >= cmp : ctk[y + 1] <= cmp));
            const float2 a = __ffma2_rn(make_float2(__uint_as_float(sv[x + y]), __uint_as_float(sv[x + y + 1])),
                                        sc2, make_float2(-lv[y], -lv[y + 1]));
            const float2 ps = make_float2(vis0 ? exp2f(a.x) : 0.f, vis1 ? exp2f(a.y) : 0.f);   // P * scale
            const float2 in = __ffma2_rn(g2, make_float2(__uint_as_float(dv[x + y]), __uint_as_float(dv[x + y + 1])),
                                         make_float2(-dl[y], -dl[y + 1]));
            const float2 ds = __fmul2_rn(ps, in);
            dsv[y] = ds.x;
            dsv[y + 1] = ds.y;
            pv[y] = ps.x * gp;                                      // g P, for dV
            pv[y + 1] = ps.y * gp;
          }
          const __nv_bfloat162 a0 = __floats2bfloat162_rn(dsv[0], dsv[1]);
          const __nv_bfloat162 a1 = __floats2bfloat162_rn(dsv[2], dsv[3]);
          ds_pk[x / 2] = *reinterpret_cast<const uint32_t*>(&a0);
          ds_pk[x / 2 + 1] = *reinterpret_cast<const uint32_t*>(&a1);
          if (kKeys) {
            const __nv_bfloat162 b0 = __floats2bfloat162_rn(pv[0], pv[1]);
            const __nv_bfloat162 b1 = __floats2bfloat162_rn(pv[2], pv[3]);
            p_pk[x / 2] = *reinterpret_cast<const uint32_t*>(&b0);
            p_pk[x / 2 + 1] = *reinterpret_cast<const uint32_t*>(&b1);
          }
        }
        };
        if (interior) chunk(std::true_type{});
        else chunk(std::false_type{});
        // bf16 results go back over the columns already consumed (16 c .. 16 c + 15)
        tmem_st16(trow + C::kColS + buf + 16 * c, ds_pk);
        if (kKeys) tmem_st16(trow + C::kColP + buf + 16 * c, p_pk);
      }
      if (!ok) break;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(C::kBarPReady + it % NBUF));
    }

    if (ok) ok = mbar_wait(bar(C::kBarODone), 0, gave_up, p.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      // 32-column pieces of the accumulators (rows = keys: dV first, then dK), dealt to the
      // warpgroups in turn
      constexpr int kPieces = (kKeys ? 2 : 1) * (D / 32);
#pragma unroll 1
      for (int piece = wg; piece < kPieces; piece += C::kRowWgs) {
        const int o = piece / (D / 32), c = piece % (D / 32);
        __nv_bfloat16* out = (__nv_bfloat16*)(kKeys ? (o == 0 ? p.dv : p.dk) : p.dq);
        const int64_t* st = kKeys ? p.ks : p.qs;
        const int64_t off = b * st[0] + hr * st[1] + (int64_t)rtok * st[2];
        uint32_t raw[32];
        tmem_ld32(trow + C::kColAcc + o * D + 32 * c, raw);   // warp-collective
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int x8 = 0; x8 < 4; ++x8) {
            float v8[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) v8[x] = __uint_as_float(raw[8 * x8 + x]);
            uint4* dst = reinterpret_cast<uint4*>(out + off + 32 * c + 8 * x8);
            if (p.accumulate) {
              const uint4 old = *dst;
              const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&old);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                v8[2 * x] += __low2float(h2[x]);
                v8[2 * x + 1] += __high2float(h2[x]);
              }
            }
            uint4 pk;
            __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
            for (int x = 0; x < 4; ++x) h2[x] = __floats2bfloat162_rn(v8[2 * x], v8[2 * x + 1]);
            *dst = pk;
          }
        }
      }
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

template <int D, int KC, int NBUF, int RW, bool TMA>
cudaError_t launch_branch_as(const BwdTcParams& p, const CUtensorMap* tm, cudaStream_t st) {
  using C0 = BCfg<D, KC, 0, NBUF, RW>;
  using C1 = BCfg<D, KC, 1, NBUF, RW>;
  cudaError_t e = cudaFuncSetAttribute(bwd_tc_kernel<D, KC, 0, NBUF, RW, TMA>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, C0::kBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bwd_tc_kernel<D, KC, 1, NBUF, RW, TMA>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, C1::kBytes);
  if (e != cudaSuccess) return e;
  bwd_tc_kernel<D, KC, 0, NBUF, RW, TMA><<<(unsigned)(p.B * p.Hq * p.n_tiles), C0::kThreads, C0::kBytes, st>>>(
      p, tm[0], tm[1], tm[2], tm[3]);
  bwd_tc_kernel<D, KC, 1, NBUF, RW, TMA><<<(unsigned)(p.B * p.Hkv * p.n_tiles), C1::kThreads, C1::kBytes, st>>>(
      p, tm[0], tm[1], tm[2], tm[3]);
  bump_launches(2);
  return cudaGetLastError();
}

// tm: tensor maps of q, k, v, dy with boxes of KC tokens when the branch's tiles come by TMA,
// else null.
template <int D, int KC, int NBUF, int RW>
cudaError_t launch_branch(const BwdTcParams& p, const CUtensorMap* tm, cudaStream_t st) {
  if (tm) return launch_branch_as<D, KC, NBUF, RW, true>(p, tm, st);
  const CUtensorMap none[4] = {};
  return launch_branch_as<D, KC, NBUF, RW, false>(p, none, st);
}

constexpr int kWideDefault = 1;   // shape for w > 128

// Kernel shape: 0 = 64-wide column tiles, one score buffer (narrow windows: least band-edge
// waste, two CTAs per SM at d = 64); 1 = 64-wide tiles, two score buffers and two row
// warpgroups (products of the next tile overlap the row work of this one); 2 = 128-wide
// tiles, one buffer, two row warpgroups (a third fewer tensor-pipe cycles per column than
// 64-wide tiles, and half the wait for the row threads).
// sa_debug_set(SA_DEBUG_SCORE_BLOCK, 64 | 128) forces shape 0 or 2.
int bwd_shape(int w) {
  const int forced = debug_option(SA_DEBUG_SCORE_BLOCK);
  if (forced) return forced == 64 ? 0 : 2;
  return w <= 128 ? 0 : kWideDefault;
}

bool bwd_tc_disabled() { return debug_option(SA_DEBUG_TENSOR_CORES) == 0; }

}  // namespace

bool tc_backward_supported(const BwdArgs& a, int dtype) {
  if (bwd_tc_disabled() || dtype != SA_BF16 || (a.d != 128 && a.d != 64)) return false;
  return a.n >= 1 && (int64_t)a.B * a.Hq * ((a.n + kTile - 1) / kTile) <= 0x3fffffff;
}

cudaError_t launch_bwd_tc(const BwdArgs& a, cudaStream_t st) {
  for (int x = 0; x < a.nbranch; ++x) {
    BwdTcParams p{};
    p.q = a.q; p.k = a.k; p.v = a.v; p.dy = a.dy;
    p.perm = x == 0 ? a.perm : nullptr;
    p.lse = a.lse_x[x];
    p.delta = a.delta + (size_t)x * a.B * a.Hq * a.n;
    p.gate_logit = a.gate_logits ? a.gate_logits + (size_t)x * a.Hq : nullptr;
    p.dq = a.dq; p.dk = a.dk; p.dv = a.dv;
    p.accumulate = x > 0;
    p.status = status_ptr();
    if (!p.status) return cudaErrorUnknown;
    p.abort_flag = a.abort_flag;
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.Hq / a.Hkv; p.n = a.n; p.w = a.w;
    const MaskGeom mg = make_geom(a.n, a.w, a.flags, x == 1);
    p.h = mg.h;
    p.causal = mg.causal; p.linear = mg.linear; p.one_sided = mg.one_sided;
    p.full_range = mg.one_sided ? (a.w - 1 >= a.n) : (2ll * mg.h + 1 >= a.n);
    p.n_tiles = (a.n + kTile - 1) / kTile;
    p.scale = a.scale;
    p.scale2 = a.scale * kLog2e;
    for (int i = 0; i < 3; ++i) { p.qs[i] = a.qs[i]; p.ks[i] = a.ks[i]; }
    const int shape = bwd_shape(a.w);
    // whole-tile TMA loads for the one-sided SWA branch (otherwise the gather serves it too)
    CUtensorMap maps[4];
    const CUtensorMap* tm = nullptr;
    const int kc = shape == 2 ? 128 : 64;
    if (x == 1 && mg.one_sided && debug_option(SA_DEBUG_SWA_TILE_LOADS) != 0 && aligned16(a.q) &&
        aligned16(a.k) && aligned16(a.v) && aligned16(a.dy) &&
        make_map_bhnd(&maps[0], a.q, a.B, a.Hq, a.n, a.d, a.qs, kc) &&
        make_map_bhnd(&maps[1], a.k, a.B, a.Hkv, a.n, a.d, a.ks, kc) &&
        make_map_bhnd(&maps[2], a.v, a.B, a.Hkv, a.n, a.d, a.ks, kc) &&
        make_map_bhnd(&maps[3], a.dy, a.B, a.Hq, a.n, a.d, a.qs, kc))
      tm = maps;
    cudaError_t e;
    if (a.d == 128)
      e = shape == 0 ? launch_branch<128, 64, 1, 1>(p, tm, st)
          : shape == 1 ? launch_branch<128, 64, 2, 2>(p, tm, st)
                       : launch_branch<128, 128, 1, 2>(p, tm, st);
    else
      e = shape == 0 ? launch_branch<64, 64, 1, 1>(p, tm, st)
          : shape == 1 ? launch_branch<64, 64, 2, 2>(p, tm, st)
                       : launch_branch<64, 128, 1, 2>(p, tm, st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace sa
