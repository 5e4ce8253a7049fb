// Entry points of the C ABI: argument checks, workspace carving, kernel choice.
// Nothing here touches device data on the host; every call only enqueues kernels.
#include <atomic>
#include <cmath>

#include "sa_common.cuh"
#include "sa_fwd_tc.cuh"

namespace sa {

__device__ int g_status_word = 0;
static std::atomic<uint64_t> g_launches{0};
static cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

void bump_launches(uint64_t k) { g_launches.fetch_add(k, std::memory_order_relaxed); }

// Test hooks: score block auto, SWA tile loads on, tensor cores on, wide gate tiles on.
static std::atomic<int> g_debug[SA_DEBUG_KEYS] = {{0}, {1}, {1}, {1}};

int debug_option(int key) {
  return key >= 0 && key < SA_DEBUG_KEYS ? g_debug[key].load(std::memory_order_relaxed) : 0;
}

int* status_ptr() {
  static std::atomic<int*> ptrs[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  int* p = ptrs[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress((void**)&p, g_status_word) != cudaSuccess) return nullptr;
    ptrs[dev].store(p, std::memory_order_release);
  }
  return p;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool good_ptr(const void* p) { return p != nullptr && aligned16(p); }

sa_status check_problem(const sa_problem* p) {
  if (!p) return SA_ERR_INVALID_ARG;
  if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->n < 1 || p->d < 1 || p->w < 1)
    return SA_ERR_INVALID_ARG;
  if (p->Hq % p->Hkv != 0) return SA_ERR_INVALID_ARG;
  if (p->dtype != SA_F32 && p->dtype != SA_BF16) return SA_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(SA_CAUSAL | SA_LINEAR_WINDOW | SA_SWA_ONE_SIDED | SA_SAVE_FOR_BWD |
                             SA_VALIDATE_PERM))
    return SA_ERR_INVALID_ARG;
  if ((p->flags & SA_SWA_ONE_SIDED) && !(p->flags & SA_CAUSAL)) return SA_ERR_INVALID_ARG;
  if (!(p->softmax_scale >= 0.f) || std::isinf(p->softmax_scale)) return SA_ERR_INVALID_ARG;
  if (p->d % 8 != 0 || p->d > 256) return SA_ERR_UNSUPPORTED;
  if (p->Hq > 65535 || p->B > 32767 || p->n > (1 << 30)) return SA_ERR_UNSUPPORTED;
  for (int i = 0; i < 3; ++i) {
    if (p->q_stride[i] < 0 || p->kv_stride[i] < 0) return SA_ERR_INVALID_ARG;
    if (p->q_stride[i] % 8 != 0 || p->kv_stride[i] % 8 != 0) return SA_ERR_INVALID_ARG;
  }
  if (p->q_stride[2] < p->d || p->kv_stride[2] < p->d) return SA_ERR_INVALID_ARG;
  return SA_OK;
}

// Bytes of one branch output in the layout of q (its strides): what the gated forward can
// use as scratch for the local branch's rows.
size_t branch_bytes(const sa_problem* p) {
  const int64_t elems = (p->B - 1) * p->q_stride[0] + (p->Hq - 1) * p->q_stride[1] +
                        (int64_t)(p->n - 1) * p->q_stride[2] + p->d;
  return (size_t)elems * (p->dtype == SA_BF16 ? 2 : 4);
}

// Bytes a tensor with the given strides spans (the rotated copies of the unfused RoPE path).
size_t span_bytes(const sa_problem* p, bool kv) {
  const int64_t* s = kv ? p->kv_stride : p->q_stride;
  const int H = kv ? p->Hkv : p->Hq;
  const int64_t elems = (p->B - 1) * s[0] + (H - 1) * s[1] + (int64_t)(p->n - 1) * s[2] + p->d;
  return ((size_t)elems * (p->dtype == SA_BF16 ? 2 : 4) + 255) / 256 * 256;
}

float scale_of(const sa_problem* p) {
  return p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / std::sqrt((float)p->d);
}

FwdArgs fwd_args(const sa_problem* p, const void* q, const void* k, const void* v, bool swa) {
  FwdArgs a{};
  a.q = q; a.k = k; a.v = v;
  a.B = p->B; a.Hq = p->Hq; a.Hkv = p->Hkv; a.n = p->n; a.d = p->d; a.w = p->w;
  a.flags = p->flags;
  a.scale = scale_of(p);
  for (int i = 0; i < 3; ++i) { a.qs[i] = p->q_stride[i]; a.ks[i] = p->kv_stride[i]; }
  a.swa = swa;
  a.abort_flag = (p->flags & SA_VALIDATE_PERM) ? status_ptr() : nullptr;
  return a;
}

// One forward branch: the tensor-core kernel when the shape qualifies, else the general one.
cudaError_t run_forward(const FwdArgs& a, int dtype, cudaStream_t st) {
  const bool prof = !a.swa && g_prof_start && g_prof_stop;
  if (prof) cudaEventRecord(g_prof_start, st);
  const cudaError_t e = tc_forward_supported(a, dtype) ? launch_fwd_tc(a, st)
                                                       : launch_fwd_simt(a, dtype, st);
  if (prof) cudaEventRecord(g_prof_stop, st);
  return e;
}

sa_status from_cuda(cudaError_t e) { return e == cudaSuccess ? SA_OK : SA_ERR_CUDA; }

sa_status maybe_validate(const sa_problem* p, const int32_t* perm, const int32_t* inv,
                         cudaStream_t st) {
  if (!(p->flags & SA_VALIDATE_PERM)) return SA_OK;
  return from_cuda(launch_validate_perm(perm, inv, p->B, p->n, st));
}

}  // namespace
}  // namespace sa

using namespace sa;

extern "C" {

void sa_problem_set_contiguous(sa_problem* p) {
  if (!p) return;
  p->q_stride[2] = p->d;
  p->q_stride[1] = (int64_t)p->n * p->d;
  p->q_stride[0] = (int64_t)p->Hq * p->n * p->d;
  p->kv_stride[2] = p->d;
  p->kv_stride[1] = (int64_t)p->n * p->d;
  p->kv_stride[0] = (int64_t)p->Hkv * p->n * p->d;
}

size_t sa_workspace_bytes(const sa_problem* p, int op) {
  if (!p) return (size_t)-1;
  switch (op) {
    case SA_OP_MAKE_PERM:
      if (p->B < 1 || p->n < 1) return (size_t)-1;
      return make_perm_ws_bytes(p->B, p->n);
    case SA_OP_COVERAGE:
      if (p->n < 1) return (size_t)-1;
      return coverage_ws_bytes(p->L, p->n);
    case SA_OP_FORWARD:
    case SA_OP_SWA_FORWARD:
    case SA_OP_GATED_FORWARD:
      return check_problem(p) == SA_OK ? 0 : (size_t)-1;
    case SA_OP_GATED_FORWARD_SCRATCH:
      return check_problem(p) == SA_OK ? branch_bytes(p) : (size_t)-1;
    case SA_OP_BACKWARD:
      if (check_problem(p) != SA_OK) return (size_t)-1;
      return bwd_ws_bytes(p->B, p->Hq, p->n, nullptr);
    case SA_OP_FORWARD_ROPE: {
      if (check_problem(p) != SA_OK || p->d % 2 != 0) return (size_t)-1;
      FwdArgs a = fwd_args(p, p, p, p, false);      // pointers unused by the support test
      if (tc_forward_supported(a, p->dtype)) return 0;
      return span_bytes(p, false) + span_bytes(p, true);
    }
    default:
      return (size_t)-1;
  }
}

sa_status sa_make_perm(uint64_t seed, uint32_t layer, int32_t B, int32_t n, int32_t* perm,
                       int32_t* inv, void* ws, size_t ws_bytes, sa_stream_t stream) {
  if (B < 1 || n < 1) return SA_ERR_INVALID_ARG;
  if (B > 32767 || n > (1 << 30)) return SA_ERR_UNSUPPORTED;
  if (!good_ptr(perm) || !good_ptr(inv) || !good_ptr(ws)) return SA_ERR_INVALID_ARG;
  if (ws_bytes < make_perm_ws_bytes(B, n)) return SA_ERR_WORKSPACE;
  return from_cuda(launch_make_perm(seed, layer, B, n, perm, inv, ws, (cudaStream_t)stream));
}

sa_status sa_forward(const sa_problem* p, const void* q, const void* k, const void* v,
                     const int32_t* perm, const int32_t* inv, void* y, float* lse, void* ws,
                     size_t ws_bytes, sa_stream_t stream) {
  (void)ws; (void)ws_bytes;
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(perm) || !good_ptr(inv) ||
      !good_ptr(y) || (lse && !aligned16(lse)))
    return SA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if ((s = maybe_validate(p, perm, inv, st)) != SA_OK) return s;
  FwdArgs a = fwd_args(p, q, k, v, false);
  a.perm = perm; a.inv = inv; a.y = y; a.lse = lse;
  return from_cuda(run_forward(a, p->dtype, st));
}

sa_status sa_swa_forward(const sa_problem* p, const void* q, const void* k, const void* v,
                         void* y, float* lse, void* ws, size_t ws_bytes, sa_stream_t stream) {
  (void)ws; (void)ws_bytes;
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(y) || (lse && !aligned16(lse)))
    return SA_ERR_INVALID_ARG;
  FwdArgs a = fwd_args(p, q, k, v, true);
  a.y = y; a.lse = lse;
  return from_cuda(run_forward(a, p->dtype, (cudaStream_t)stream));
}

sa_status sa_swa_gated_forward(const sa_problem* p, const void* q, const void* k,
                               const void* v, const int32_t* perm, const int32_t* inv,
                               const float* gate_logits, void* y, void* y_sa, void* y_swa,
                               float* lse_sa, float* lse_swa, void* ws, size_t ws_bytes,
                               sa_stream_t stream) {
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(perm) || !good_ptr(inv) ||
      !good_ptr(y) || !gate_logits)
    return SA_ERR_INVALID_ARG;
  if (ws && !aligned16(ws)) return SA_ERR_INVALID_ARG;
  if ((y_sa && !aligned16(y_sa)) || (y_swa && !aligned16(y_swa)) ||
      (lse_sa && !aligned16(lse_sa)) || (lse_swa && !aligned16(lse_swa)))
    return SA_ERR_INVALID_ARG;
  if ((p->flags & SA_SAVE_FOR_BWD) && (!y_sa || !y_swa || !lse_sa || !lse_swa))
    return SA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if ((s = maybe_validate(p, perm, inv, st)) != SA_OK) return s;
  // Two launches.  The SA branch first: its ungated rows land in y_sa, else in the scratch,
  // else in y itself.  The local branch then owns each output row exactly once and its rows
  // are consecutive tokens, so the matching SA rows are read back as contiguous runs, both
  // gates are applied and y is written: by the two warps that have nothing to load when the
  // local branch's tiles come by TMA (this needs a home for the local rows other than the
  // buffer the SA rows sit in: y_swa, or y when the SA rows are elsewhere), otherwise in the
  // row threads' epilogue.  (Reading the scattered rows of the local branch from the SA
  // branch's epilogue, the other possible order, costs more than a third launch would.)
  const bool scratch = ws && ws_bytes >= branch_bytes(p);
  void* sa_rows = y_sa ? y_sa : (scratch ? ws : y);
  FwdArgs a = fwd_args(p, q, k, v, false);
  a.perm = perm; a.inv = inv; a.y = sa_rows; a.lse = lse_sa;
  cudaError_t e = run_forward(a, p->dtype, st);
  if (e != cudaSuccess) return SA_ERR_CUDA;
  FwdArgs b = fwd_args(p, q, k, v, true);
  b.y = y; b.y_branch = y_swa; b.lse = lse_swa;
  b.y_other = sa_rows; b.gate_logits = gate_logits;
  return from_cuda(run_forward(b, p->dtype, st));
}

sa_status sa_rope_apply(const sa_problem* p, int32_t kv, const void* x, const float* rope_cos,
                        const float* rope_sin, int32_t inverse, void* out, sa_stream_t stream) {
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (p->d % 2 != 0 || !good_ptr(x) || !good_ptr(out) || !rope_cos || !rope_sin)
    return SA_ERR_INVALID_ARG;
  return from_cuda(launch_rope_apply(x, out, p->B, kv ? p->Hkv : p->Hq, p->n, p->d,
                                     kv ? p->kv_stride : p->q_stride, p->dtype, rope_cos,
                                     rope_sin, inverse != 0, (cudaStream_t)stream));
}

namespace {
// Where the fused rotation does not apply: rotated copies of q and k in the workspace.
sa_status rope_prepass(const sa_problem* p, const void*& q, const void*& k, const float* rope_cos,
                       const float* rope_sin, void* ws, size_t ws_bytes, cudaStream_t st) {
  const size_t qb = span_bytes(p, false), kb = span_bytes(p, true);
  if (!ws || !aligned16(ws)) return SA_ERR_INVALID_ARG;
  if (ws_bytes < qb + kb) return SA_ERR_WORKSPACE;
  void* qr = ws;
  void* kr = (char*)ws + qb;
  if (launch_rope_apply(q, qr, p->B, p->Hq, p->n, p->d, p->q_stride, p->dtype, rope_cos, rope_sin,
                        false, st) != cudaSuccess ||
      launch_rope_apply(k, kr, p->B, p->Hkv, p->n, p->d, p->kv_stride, p->dtype, rope_cos,
                        rope_sin, false, st) != cudaSuccess)
    return SA_ERR_CUDA;
  q = qr;
  k = kr;
  return SA_OK;
}
}  // namespace

sa_status sa_forward_rope(const sa_problem* p, const void* q, const void* k, const void* v,
                          const int32_t* perm, const int32_t* inv, const float* rope_cos,
                          const float* rope_sin, void* y, float* lse, void* ws, size_t ws_bytes,
                          sa_stream_t stream) {
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (p->d % 2 != 0 || !rope_cos || !rope_sin || !aligned16(rope_cos) || !aligned16(rope_sin))
    return SA_ERR_INVALID_ARG;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(perm) || !good_ptr(inv) ||
      !good_ptr(y) || (lse && !aligned16(lse)))
    return SA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if ((s = maybe_validate(p, perm, inv, st)) != SA_OK) return s;
  FwdArgs a = fwd_args(p, q, k, v, false);
  a.perm = perm; a.inv = inv; a.y = y; a.lse = lse;
  if (tc_forward_supported(a, p->dtype)) {
    a.rope_cos = rope_cos; a.rope_sin = rope_sin;
  } else {
    if ((s = rope_prepass(p, a.q, a.k, rope_cos, rope_sin, ws, ws_bytes, st)) != SA_OK) return s;
  }
  return from_cuda(run_forward(a, p->dtype, st));
}

sa_status sa_swa_gated_forward_rope(const sa_problem* p, const void* q, const void* k,
                                    const void* v, const int32_t* perm, const int32_t* inv,
                                    const float* rope_cos, const float* rope_sin,
                                    const float* gate_logits, void* y, void* y_sa, void* y_swa,
                                    float* lse_sa, float* lse_swa, void* ws, size_t ws_bytes,
                                    sa_stream_t stream) {
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (p->d % 2 != 0 || !rope_cos || !rope_sin || !aligned16(rope_cos) || !aligned16(rope_sin))
    return SA_ERR_INVALID_ARG;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(perm) || !good_ptr(inv) ||
      !good_ptr(y) || !gate_logits)
    return SA_ERR_INVALID_ARG;
  if ((y_sa && !aligned16(y_sa)) || (y_swa && !aligned16(y_swa)) ||
      (lse_sa && !aligned16(lse_sa)) || (lse_swa && !aligned16(lse_swa)))
    return SA_ERR_INVALID_ARG;
  if ((p->flags & SA_SAVE_FOR_BWD) && (!y_sa || !y_swa || !lse_sa || !lse_swa))
    return SA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if ((s = maybe_validate(p, perm, inv, st)) != SA_OK) return s;
  FwdArgs probe = fwd_args(p, q, k, v, false);
  const bool fused = tc_forward_supported(probe, p->dtype);
  if (!fused && (s = rope_prepass(p, q, k, rope_cos, rope_sin, ws, ws_bytes, st)) != SA_OK)
    return s;
  // SA branch first, the local branch combines (see sa_swa_gated_forward)
  void* sa_rows = y_sa ? y_sa : y;
  FwdArgs a = fwd_args(p, q, k, v, false);
  a.perm = perm; a.inv = inv; a.y = sa_rows; a.lse = lse_sa;
  if (fused) { a.rope_cos = rope_cos; a.rope_sin = rope_sin; }
  if (run_forward(a, p->dtype, st) != cudaSuccess) return SA_ERR_CUDA;
  FwdArgs b = fwd_args(p, q, k, v, true);
  b.y = y; b.y_branch = y_swa; b.lse = lse_swa;
  b.y_other = sa_rows; b.gate_logits = gate_logits;
  if (fused) { b.rope_cos = rope_cos; b.rope_sin = rope_sin; }
  return from_cuda(run_forward(b, p->dtype, st));
}

sa_status sa_backward(const sa_problem* p, const void* q, const void* k, const void* v,
                      const int32_t* perm, const int32_t* inv, const float* gate_logits,
                      const void* y_sa, const void* y_swa, const float* lse_sa,
                      const float* lse_swa, const void* dy, void* dq, void* dk, void* dv,
                      float* dgate_logits, void* ws, size_t ws_bytes, sa_stream_t stream) {
  sa_status s = check_problem(p);
  if (s != SA_OK) return s;
  if (!good_ptr(q) || !good_ptr(k) || !good_ptr(v) || !good_ptr(perm) || !good_ptr(inv) ||
      !good_ptr(y_sa) || !good_ptr(lse_sa) || !good_ptr(dy) || !good_ptr(dq) || !good_ptr(dk) ||
      !good_ptr(dv) || !good_ptr(ws))
    return SA_ERR_INVALID_ARG;
  if (gate_logits && (!good_ptr(y_swa) || !good_ptr(lse_swa) || !dgate_logits))
    return SA_ERR_INVALID_ARG;
  int chunks = 0;
  if (ws_bytes < bwd_ws_bytes(p->B, p->Hq, p->n, &chunks)) return SA_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  if ((s = maybe_validate(p, perm, inv, st)) != SA_OK) return s;
  BwdArgs a{};
  a.q = q; a.k = k; a.v = v; a.dy = dy; a.perm = perm; a.inv = inv;
  a.gate_logits = gate_logits;
  a.y_x[0] = y_sa; a.y_x[1] = y_swa; a.lse_x[0] = lse_sa; a.lse_x[1] = lse_swa;
  a.dq = dq; a.dk = dk; a.dv = dv; a.dgate = dgate_logits;
  a.delta = (float*)ws;
  const size_t delta_bytes = ((size_t)2 * p->B * p->Hq * p->n * sizeof(float) + 255) / 256 * 256;
  a.partials = (float*)((char*)ws + delta_bytes);
  a.chunks = chunks;
  a.B = p->B; a.Hq = p->Hq; a.Hkv = p->Hkv; a.n = p->n; a.d = p->d; a.w = p->w;
  a.flags = p->flags; a.scale = scale_of(p);
  for (int i = 0; i < 3; ++i) { a.qs[i] = p->q_stride[i]; a.ks[i] = p->kv_stride[i]; }
  a.nbranch = gate_logits ? 2 : 1;
  a.abort_flag = (p->flags & SA_VALIDATE_PERM) ? status_ptr() : nullptr;
  return from_cuda(launch_bwd_simt(a, p->dtype, st));
}

sa_status sa_coverage(int32_t L, int32_t n, int32_t w, uint32_t flags, const int32_t* perm,
                      const int32_t* inv, int32_t src, int64_t* nnz, int32_t* row_count,
                      int32_t* reach, void* ws, size_t ws_bytes, sa_stream_t stream) {
  if (L < 1 || n < 1 || w < 1 || src < 0 || src >= n) return SA_ERR_INVALID_ARG;
  if (n > (1 << 30)) return SA_ERR_UNSUPPORTED;
  if (flags & ~(uint32_t)(SA_CAUSAL | SA_LINEAR_WINDOW)) return SA_ERR_INVALID_ARG;
  if (!good_ptr(perm) || !good_ptr(inv) || !nnz || !reach || !good_ptr(ws))
    return SA_ERR_INVALID_ARG;
  if (ws_bytes < coverage_ws_bytes(L, n)) return SA_ERR_WORKSPACE;
  return from_cuda(launch_coverage(L, n, w, flags, perm, inv, src, nnz, row_count, reach, ws,
                                   (cudaStream_t)stream));
}

sa_status sa_read_status(sa_stream_t stream) {
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SA_ERR_CUDA;
  int* p = status_ptr();
  if (!p) return SA_ERR_CUDA;
  int host = 0;
  if (cudaMemcpy(&host, p, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SA_ERR_CUDA;
  if (host != 0) {
    const int zero = 0;
    if (cudaMemcpy(p, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess)
      return SA_ERR_CUDA;
  }
  return (sa_status)host;
}

const char* sa_status_string(sa_status s) {
  switch (s) {
    case SA_OK: return "ok";
    case SA_ERR_INVALID_ARG: return "invalid argument";
    case SA_ERR_UNSUPPORTED: return "unsupported shape or option";
    case SA_ERR_WORKSPACE: return "workspace too small";
    case SA_ERR_CUDA: return "CUDA runtime error";
    case SA_ERR_BAD_PERM: return "perm/inv are not mutually inverse permutations";
    case SA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case SA_ERR_TOO_LARGE: return "B*n needs more scratch than sa_make_perm_static has built in";
    default: return "unknown status";
  }
}

void sa_set_profile_events(void* start, void* stop) {
  g_prof_start = (cudaEvent_t)start;
  g_prof_stop = (cudaEvent_t)stop;
}

uint64_t sa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

sa_status sa_debug_set(int key, int value) {
  if (key < 0 || key >= SA_DEBUG_KEYS) return SA_ERR_INVALID_ARG;
  if (key == SA_DEBUG_SCORE_BLOCK ? (value != 0 && value != 64 && value != 128)
                                  : (value != 0 && value != 1))
    return SA_ERR_INVALID_ARG;
  g_debug[key].store(value, std::memory_order_relaxed);
  return SA_OK;
}

}  // extern "C"
