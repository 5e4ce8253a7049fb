/*
 * sa.h -- C ABI of the Stochastic Attention (SA) hot path for NVIDIA B200 (sm_100a).
 *
 * The operation (paper Sec. 3.3, Alg. 1, Eq. 3/4; App. B "Stochastic attention mask"):
 * draw a uniform random permutation sigma of the n tokens of a sequence, run softmax
 * sliding-window attention of width w in the permuted order, and put the result back
 * in the original order.  In the original order, query token i sees key token j iff
 *
 *     2 * dist(inv[i], inv[j]) < w        (window in shuffled space, Eq. 3)
 *     and, with SA_CAUSAL,  j <= i        (causality in ORIGINAL space, App. B)
 *
 * where inv[i] is the slot of token i (the paper's sigma(i)), perm[p] the token in
 * slot p, and dist is the circular distance |a-b|_n = min(|a-b|, n-|a-b|) of Sec. 3.1
 * (plain |a-b| with SA_LINEAR_WINDOW).  The gated form (Sec. 3.4, Eq. 5, Alg. 2) adds
 * an ordinary sliding-window branch: y = sig(l_sa) y_sa + sig(l_swa) y_swa, with two
 * independent sigmoids and, in this library, one scalar logit per head and branch.
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer unless a comment says "host".  The caller owns
 *     every buffer, workspace included; the library allocates nothing and frees nothing.
 *   - Work is only enqueued on the caller's stream; no call synchronises except
 *     sa_read_status.  Inputs are never written.
 *   - Tensors: q, y, dq, dy, y_sa, y_swa are [B,Hq,n,d]; k, v, dk, dv are [B,Hkv,n,d];
 *     addressed through the element strides in sa_problem (d is contiguous).  perm and
 *     inv are contiguous int32 [B,n]; lse_* contiguous fp32 [B,Hq,n]; gate logits
 *     contiguous fp32 [2,Hq] (row 0 = SA branch, row 1 = SWA branch).
 *   - Everything the caller sees is in ORIGINAL token order.
 *   - Query head hq reads KV head hq / (Hq/Hkv) (contiguous GQA groups).
 *   - Data pointers must be 16-byte aligned and all strides multiples of 8 elements.
 *   - Errors the host can see (bad shapes, null or misaligned pointers, short
 *     workspace) return a code before anything is launched.  Errors only the device can
 *     see (SA_VALIDATE_PERM found a non-bijection, a bounded wait ran out) are recorded
 *     in a device status word that sa_read_status returns; the kernel then returns
 *     normally and its outputs are unspecified.  Nothing traps.  The word is sticky: once
 *     it holds SA_ERR_TIMEOUT, later tensor-core launches return at once without writing
 *     their outputs until sa_read_status has been called (which clears it).
 */
#ifndef SA_B200_SA_H_
#define SA_B200_SA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* sa_stream_t; /* a cudaStream_t; NULL = the legacy default stream */

typedef enum {
  SA_OK = 0,
  SA_ERR_INVALID_ARG = 1, /* null/misaligned pointer, bad shape or stride               */
  SA_ERR_UNSUPPORTED = 2, /* valid request this build has no kernel for                 */
  SA_ERR_WORKSPACE = 3,   /* ws_bytes smaller than sa_workspace_bytes()                  */
  SA_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error, no device)       */
  SA_ERR_BAD_PERM = 5,    /* device: perm/inv are not mutually inverse bijections       */
  SA_ERR_TIMEOUT = 6,     /* device: a bounded wait inside a kernel ran out             */
  SA_ERR_TOO_LARGE = 7    /* sa_make_perm_static: B, n need more than the built-in scratch */
} sa_status;

typedef enum { SA_F32 = 0, SA_BF16 = 1 } sa_dtype;

enum {
  SA_CAUSAL = 1,        /* j <= i in the original order (Sec. 3.3 causal paragraph; App. B)   */
  SA_LINEAR_WINDOW = 2, /* plain |a-b| between slots; default is circular |a-b|_n (Sec. 3.1) */
  SA_SWA_ONE_SIDED = 4, /* the SWA branch uses {j : 0 <= i-j <= w-1} (Sec. 3.1 footnote);    */
                        /* without it the SWA branch is the SA rule under the identity       */
  SA_SAVE_FOR_BWD = 8,  /* gated forward: y_sa, y_swa, lse_sa, lse_swa must all be given     */
  SA_VALIDATE_PERM = 16 /* check on the device that inv[perm[p]] == p, 0 <= perm[p] < n      */
};

typedef enum {
  SA_OP_MAKE_PERM = 0,
  SA_OP_FORWARD = 1,
  SA_OP_SWA_FORWARD = 2,
  SA_OP_GATED_FORWARD = 3,
  SA_OP_BACKWARD = 4,
  SA_OP_COVERAGE = 5,
  SA_OP_GATED_FORWARD_SCRATCH = 6, /* optional scratch of sa_swa_gated_forward, see there */
  SA_OP_FORWARD_ROPE = 7           /* sa_forward_rope / sa_swa_gated_forward_rope           */
} sa_op;

typedef struct {
  int32_t B, Hq, Hkv;  /* batch, query heads, KV heads; Hq % Hkv == 0                     */
  int32_t n, d, w;     /* tokens, head dim (multiple of 8, <= 256), window width (>= 1)   */
  int32_t dtype;       /* sa_dtype of q/k/v/y/dy/dq/dk/dv                                 */
  uint32_t flags;      /* SA_* bits                                                       */
  float softmax_scale; /* multiplies q.k (Eq. 1); 0 selects 1/sqrt(d)                     */
  int32_t L;           /* layers, used by SA_OP_COVERAGE sizing only; else ignored        */
  int64_t q_stride[3];  /* element strides of q, y, dq, dy, y_sa, y_swa: batch, head, token */
  int64_t kv_stride[3]; /* element strides of k, v, dk, dv: batch, head, token            */
} sa_problem;

/* Fills the two stride triples for contiguous [B,H,n,d] tensors.  Host-only helper. */
void sa_problem_set_contiguous(sa_problem* p);

/* Bytes of workspace the given operation needs for this problem (0 is possible; then
 * ws may be NULL).  Only B, n matter for SA_OP_MAKE_PERM; L, n for SA_OP_COVERAGE.
 * Returns (size_t)-1 for an invalid problem. */
size_t sa_workspace_bytes(const sa_problem* p, int op);

/* Alg. 1 line 1: one uniform random permutation per sequence and its inverse.
 * Sequence b, token i gets the 64-bit key formed by the first two output words of
 * Philox4x32-10 with counter (i, b, layer, 0) and key (seed low word, seed high word);
 * perm[b,:] lists the tokens in increasing (key, token) order; inv[b, perm[b,p]] = p.
 * A pure function of (seed, layer, b, n): any process regenerates the same sigma.
 * perm, inv: out, int32 [B,n].  ws: scratch of sa_workspace_bytes(.., SA_OP_MAKE_PERM). */
sa_status sa_make_perm(uint64_t seed, uint32_t layer, int32_t B, int32_t n, int32_t* perm,
                       int32_t* inv, void* ws, size_t ws_bytes, sa_stream_t stream);

/* sa_make_perm for callers that cannot allocate device memory.  The paper has no counterpart:
 * this is the same operation as sa_make_perm with the same result, bit for bit; only the home
 * of the sort's scratch differs.  It is meant for code that runs where cudaMalloc (or a
 * framework's caching allocator) is off limits -- a hook called while another library holds
 * the allocator, a real-time loop that must not touch the driver's memory manager, a plug-in
 * that is handed output buffers and nothing else -- and so cannot provide the workspace that
 * sa_make_perm asks for.  The scratch lives inside the library image instead: a fixed array of
 * SA_STATIC_SCRATCH_BYTES that every GPU which loads the library holds until the process exits.
 *   - perm, inv: out, device, int32 [B,n], 16-byte aligned, owned by the caller as always.
 *   - Limit: sa_workspace_bytes(.., SA_OP_MAKE_PERM) for (B, n) must not exceed
 *     SA_STATIC_SCRATCH_BYTES (about 200,000 tokens in total, B*n); beyond that the call
 *     returns SA_ERR_TOO_LARGE and launches nothing.
 *   - The call allocates and frees nothing, and only enqueues kernels on `stream`.
 *   - The first call on each device looks up the array's device address (one runtime query,
 *     with that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left.
 *     The only part that must start at zero (the sort's bucket counters) is cleared by
 *     each call on its stream; everything else is written before it is read.  Two
 *     calls whose kernels may run at the same time on one GPU (different streams, or
 *     different host threads) race on the array and give wrong permutations: keep the
 *     calls of a device on one stream, or order them yourself. */
#define SA_STATIC_SCRATCH_BYTES (4u << 20)
sa_status sa_make_perm_static(uint64_t seed, uint32_t layer, int32_t B, int32_t n,
                              int32_t* perm, int32_t* inv, sa_stream_t stream);

/* SA forward (Alg. 1; Eq. 1 on the neighbourhood of Eq. 3; mask of App. B).
 * Rows of q/k/v are gathered through perm inside the kernel and rows of y are scattered
 * back; no permuted copy of any tensor is made.  y: out.  lse: out, nullable, the
 * log-sum-exp of each query's visible scaled scores (needed by sa_backward). */
sa_status sa_forward(const sa_problem* p, const void* q, const void* k, const void* v,
                     const int32_t* perm, const int32_t* inv, void* y, float* lse, void* ws,
                     size_t ws_bytes, sa_stream_t stream);

/* Plain sliding-window attention in the original order (Eq. 1): the local branch of the
 * gated form and the baseline the permutation overhead is measured against. */
sa_status sa_swa_forward(const sa_problem* p, const void* q, const void* k, const void* v,
                         void* y, float* lse, void* ws, size_t ws_bytes, sa_stream_t stream);

/* Gated SA + SWA forward (Alg. 2, Eq. 5) with per-head scalar gates:
 * y = sigmoid(gate_logits[0,hq]) * y_sa + sigmoid(gate_logits[1,hq]) * y_swa.
 * y: out.  y_sa, y_swa, lse_sa, lse_swa: out, nullable unless SA_SAVE_FOR_BWD; the
 * branch outputs are stored in the run dtype before they are combined.
 * Two launches: the SA branch writes its ungated rows (to y_sa, else to ws, else to y itself),
 * then the local branch, whose rows are consecutive tokens, reads them back, applies both
 * gates and writes y.  ws is optional (sa_workspace_bytes(.., SA_OP_GATED_FORWARD) is 0): with
 * at least sa_workspace_bytes(.., SA_OP_GATED_FORWARD_SCRATCH) bytes (one branch output in
 * q's layout) a caller that keeps neither branch output still gets the faster form of the
 * combination, in which the local branch stores its rows (rounded to the run dtype) and two
 * otherwise idle warps of the same launch combine them; without any such buffer the row
 * threads combine in their epilogue, from unrounded local rows. */
sa_status sa_swa_gated_forward(const sa_problem* p, const void* q, const void* k,
                               const void* v, const int32_t* perm, const int32_t* inv,
                               const float* gate_logits, void* y, void* y_sa, void* y_swa,
                               float* lse_sa, float* lse_swa, void* ws, size_t ws_bytes,
                               sa_stream_t stream);

/* sa_make_perm + sa_swa_gated_forward (Alg. 1 line 1, Alg. 2, Eq. 5) for tensors that live in
 * HOST memory: q, k, v, y are host pointers to contiguous [B,H,n,d] tensors of p->dtype
 * (p's stride fields are ignored), gate_logits a host pointer to fp32 [2,Hq]; pinned memory
 * lets the copies overlap the kernels, pageable memory works but serialises.  The KV heads
 * travel through the GPU in n_groups contiguous ranges (the first and the last range, when
 * they hold one KV head, in q_parts ranges of its query heads if those divide evenly: the
 * ends of the pipeline are what cannot overlap), on three internal streams: copy in,
 * compute, copy out.  The permutation is drawn from (seed, layer) as in sa_make_perm and
 * shared by all ranges; every range is one sa_swa_gated_forward call given scratch, so the
 * result has the bits of that call.
 *   ws: DEVICE workspace of sa_host_forward_ws_bytes(p) bytes, 256-byte aligned, owned by the
 *       caller (device copies of q, k, v, y, one branch output, the permutation and its
 *       scratch).  No device memory is allocated; the first call on a device creates the
 *       three streams and the events of the pipeline and keeps them.
 *   stream: the call is ordered after what `stream` has queued, and `stream` waits for the
 *       last copy out, so the caller synchronises (or times) on `stream` alone.  y must not
 *       be read on the host before that.  Calls on one device must not overlap.
 * Errors: SA_ERR_INVALID_ARG, SA_ERR_WORKSPACE, SA_ERR_CUDA, and those of the two calls. */
size_t sa_host_forward_ws_bytes(const sa_problem* p);
sa_status sa_swa_gated_forward_host(const sa_problem* p, const void* q, const void* k,
                                    const void* v, const float* gate_logits, void* y,
                                    uint64_t seed, uint32_t layer, int32_t n_groups,
                                    int32_t q_parts, void* ws, size_t ws_bytes,
                                    sa_stream_t stream);
/* The head ranges sa_swa_gated_forward_host uses, for inspection (host only, no GPU needed):
 * writes up to max_pieces rows of (kv_begin, kv_end, q_begin, q_end, carries_kv) and returns
 * their number, or -1 for bad head counts or too small an array. */
int32_t sa_host_forward_plan(int32_t Hq, int32_t Hkv, int32_t n_groups, int32_t q_parts,
                             int32_t* pieces, int32_t max_pieces);

/* Rotary position embedding with ORIGINAL token positions.  The paper applies RoPE to Q and K
 * before the shuffle, with the positions the tokens have in the sequence, not the slots they
 * are shuffled to (Sec. 4.2; attention paragraph of App. B).  Dimension c of the first half of
 * a head is paired with dimension c + d/2 (the half-split layout of the Qwen3 / Llama family);
 * token t turns the pair (x1, x2) by the angle t * base^(-2c/d):
 *     out1 = x1 cos - x2 sin,   out2 = x2 cos + x1 sin      (fp32, rounded once to the dtype).
 *
 * sa_rope_table: rope_cos, rope_sin: out, device, fp32 [n, d/2]: cosine and sine of those
 *   angles (angles in float64).  d even.
 * sa_rope_apply: the rotation as a pass of its own.  x, out: device, [B,H,n,d] with the strides
 *   of q (kv == 0: H = Hq) or of k (kv != 0: H = Hkv); out may be x.  inverse != 0 turns by the
 *   opposite angle (the transpose: maps a gradient with respect to the rotated tensor back).
 * sa_forward_rope / sa_swa_gated_forward_rope: sa_forward / sa_swa_gated_forward on rotated Q
 *   and K without that pass: bf16 with d = 64 or 128 rotates the rows inside the kernels' row
 *   gather, where the token a row belongs to is at hand (no rotated copy of Q or K exists);
 *   every other case rotates Q and K into ws first (sa_workspace_bytes(.., SA_OP_FORWARD_ROPE)
 *   bytes; 0 when the fused path applies).  Same results as sa_rope_apply followed by the plain
 *   call.  For the backward pass rotate q and k with sa_rope_apply, call sa_backward on them, and
 *   turn dq and dk back with inverse = 1.
 * Errors: as the plain calls, plus SA_ERR_INVALID_ARG for null tables or odd d. */
sa_status sa_rope_table(int32_t n, int32_t d, double base, float* rope_cos, float* rope_sin,
                        sa_stream_t stream);
sa_status sa_rope_apply(const sa_problem* p, int32_t kv, const void* x, const float* rope_cos,
                        const float* rope_sin, int32_t inverse, void* out, sa_stream_t stream);
sa_status sa_forward_rope(const sa_problem* p, const void* q, const void* k, const void* v,
                          const int32_t* perm, const int32_t* inv, const float* rope_cos,
                          const float* rope_sin, void* y, float* lse, void* ws, size_t ws_bytes,
                          sa_stream_t stream);
sa_status sa_swa_gated_forward_rope(const sa_problem* p, const void* q, const void* k,
                                    const void* v, const int32_t* perm, const int32_t* inv,
                                    const float* rope_cos, const float* rope_sin,
                                    const float* gate_logits, void* y, void* y_sa, void* y_swa,
                                    float* lse_sa, float* lse_swa, void* ws, size_t ws_bytes,
                                    sa_stream_t stream);

/* Backward of sa_forward (gate_logits == NULL: y_swa, lse_swa, dgate_logits ignored, y_sa
 * is the forward's y) or of sa_swa_gated_forward.  The paper only times this pass
 * (Sec. 4.3); the formulas are the derivative of Eq. 1 / Eq. 5 with sigma constant:
 *   P_ij = exp(scale q_i.k_j - lse_i), D_i = dY_x[i].Y_x[i], dV_j += P_ij dY_x[i],
 *   dS_ij = P_ij (dY_x[i].V_j - D_i), dQ_i += scale dS_ij K_j, dK_j += scale dS_ij Q_i,
 * per branch x with dY_x = g_x dY; dk, dv are summed over the query heads of a group;
 * dgate_logits[x,hq] = g_x (1 - g_x) sum_{b,i,c} dY Y_x.   dq, dk, dv, dgate_logits: out. */
sa_status sa_backward(const sa_problem* p, const void* q, const void* k, const void* v,
                      const int32_t* perm, const int32_t* inv, const float* gate_logits,
                      const void* y_sa, const void* y_swa, const float* lse_sa,
                      const float* lse_swa, const void* dy, void* dq, void* dk, void* dv,
                      float* dgate_logits, void* ws, size_t ws_bytes, sa_stream_t stream);

/* Mask statistics over L layers, each with its own permutation (perm, inv int32 [L,n]):
 * row_count[l,i] = number of keys query i sees at layer l (nullable), nnz[l] = their sum
 * (int64 [L]); reach[l] = |R_{l+1}(src)|, the set reachable from token src through layers
 * 0..l (Prop. 2: R_0 = {src}, R_{l+1} = union of the visible sets of R_l's members).
 * Only n, w and the mask bits of flags are used. */
sa_status sa_coverage(int32_t L, int32_t n, int32_t w, uint32_t flags, const int32_t* perm,
                      const int32_t* inv, int32_t src, int64_t* nnz, int32_t* row_count,
                      int32_t* reach, void* ws, size_t ws_bytes, sa_stream_t stream);

/* Projection gates of Eq. 5-6 (dual path) and of the single-path attention gate of App. B:
 *   out = sigmoid(y_sa w_sa^T) * y_sa  [+ sigmoid(y_swa w_swa^T) * y_swa],
 * per token and per dimension, the two sigmoids independent.  y_sa, y_swa, out: device,
 * [rows, dm] in the run dtype, row r starting ld_y (ld_out) elements after row r-1: the
 * attention outputs with the heads of a token side by side (sa_forward writes that layout
 * when given the strides of a [B,n,Hq,d] tensor).  w_sa, w_swa: device, [dm, dm] row-major
 * (out_features x in_features, a bias-free linear layer), same dtype.  y_swa == NULL selects
 * the single-path gate (w_swa ignored).  Products accumulate in fp32; the logistic and the
 * combination are fp32, rounded once to the run dtype.  dtype SA_BF16 with dm a multiple of
 * 64 and 16-byte aligned rows runs on the tensor cores; every other case on a plain kernel.
 * Nothing is allocated; inputs are not modified; out may not alias an input.
 * Errors: SA_ERR_INVALID_ARG (null pointer, rows < 1, dm < 1, ld < dm), SA_ERR_CUDA. */
sa_status sa_gate_projection_forward(int64_t rows, int32_t dm, int32_t dtype, const void* y_sa,
                                     const void* y_swa, int64_t ld_y, const void* w_sa,
                                     const void* w_swa, void* out, int64_t ld_out,
                                     sa_stream_t stream);

/* Backward of sa_gate_projection_forward.  With z = y w^T, g = sigmoid(z) per path:
 *   dz = dout * y * g * (1 - g),   dw = dz^T y,   dy = dout * g + dz w.
 * dout: device, [rows, dm], pitch ld_dout: gradient of the forward's out.  y_*, w_*: as in the
 * forward (y pitch ld_y).  dy_sa, dy_swa: out, [rows, dm], pitch ld_dy; dw_sa, dw_swa: out,
 * [dm, dm] contiguous, the sum over all rows (not accumulated into).  y_swa == NULL: single
 * path, the swa arguments are ignored.  ws: device scratch of
 * sa_gate_projection_backward_ws_bytes(rows, dm) bytes (dz and dout * g of one path at a
 * time).  bf16 with dm a multiple of 64 and 16-byte aligned rows runs three tensor-core
 * products per path (dz and dout * g are kept in bf16 between them); every other case runs
 * plain kernels with fp32 scratch.  Nothing is allocated; outputs may not alias inputs.
 * Errors: SA_ERR_INVALID_ARG, SA_ERR_WORKSPACE, SA_ERR_UNSUPPORTED, SA_ERR_CUDA. */
size_t sa_gate_projection_backward_ws_bytes(int64_t rows, int32_t dm);
sa_status sa_gate_projection_backward(int64_t rows, int32_t dm, int32_t dtype, const void* dout,
                                      int64_t ld_dout, const void* y_sa, const void* y_swa,
                                      int64_t ld_y, const void* w_sa, const void* w_swa,
                                      void* dy_sa, void* dy_swa, int64_t ld_dy, void* dw_sa,
                                      void* dw_swa, void* ws, size_t ws_bytes,
                                      sa_stream_t stream);

/* Synchronises the stream, returns the device status word (SA_OK, SA_ERR_BAD_PERM or
 * SA_ERR_TIMEOUT) of the current device and clears it. */
sa_status sa_read_status(sa_stream_t stream);

/* Static, human-readable name of a status code.  Host pointer. */
const char* sa_status_string(sa_status s);

/* Profiling hook.  start/stop are cudaEvent_t handles (host values) or both NULL.  While set,
 * every SA-branch attention kernel launched by sa_forward / sa_swa_gated_forward is bracketed
 * by cudaEventRecord(start) and cudaEventRecord(stop) on the call's stream, so a caller can
 * time that one kernel inside a longer step.  Process-wide; not thread-safe.  The paper has
 * no counterpart: this exists for the roofline measurement only. */
void sa_set_profile_events(void* start, void* stop);

/* Number of kernel launches this process has enqueued through the library so far
 * (all entry points together); used by the benchmark's launch count. */
uint64_t sa_launch_count(void);

/* Test hooks.  The library reads no environment variable; these process-wide switches exist
 * so that tests can run every kernel variant on one input.  The paper has no counterpart.
 *   SA_DEBUG_SCORE_BLOCK      0 = choose by w (default), 64 or 128 = force that score-block
 *                             width in the tensor-core forward and the matching backward shape
 *   SA_DEBUG_SWA_TILE_LOADS   1 = one-sided SWA branch loads whole tiles by TMA when the layout
 *                             allows (default), 0 = always gather rows
 *   SA_DEBUG_TENSOR_CORES     1 = tensor-core kernels where they apply (default), 0 = the
 *                             general CUDA-core kernels everywhere
 *   SA_DEBUG_GATE_WIDE_TILES  1 = 128 x 256 tiles for large gate projections (default), 0 = the
 *                             fused 128 x 128 kernel
 * Returns SA_ERR_INVALID_ARG for an unknown key or value.  Takes effect for later calls. */
typedef enum {
  SA_DEBUG_SCORE_BLOCK = 0,
  SA_DEBUG_SWA_TILE_LOADS = 1,
  SA_DEBUG_TENSOR_CORES = 2,
  SA_DEBUG_GATE_WIDE_TILES = 3,
  SA_DEBUG_KEYS = 4
} sa_debug_key;
sa_status sa_debug_set(int key, int value);

/* Test hook for the failure path of the kernels' bounded waits.  Launches one small CTA on
 * `stream` that waits, with the same wait routine the attention kernels use, on a barrier that
 * nothing ever completes, for at most limit_cycles SM clock cycles (1 .. 2^31; a million is
 * about half a millisecond).  The wait gives up, records SA_ERR_TIMEOUT in the device status
 * word and the kernel returns normally: nothing traps, faults or spins without a bound.
 * While the status word holds SA_ERR_TIMEOUT every tensor-core kernel of the library returns
 * at once without writing its outputs; sa_read_status returns the code and clears it. */
sa_status sa_debug_wait_timeout(int64_t limit_cycles, sa_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* SA_B200_SA_H_ */
