// Gated SA + SWA forward for tensors that live in HOST memory (Alg. 2 / Eq. 5 end to end:
// fresh permutation, both branches, gates), as one C-ABI call.
//
// The attention of one KV head (and of the query heads that share it) reads nothing of the
// other heads, so the heads travel through the GPU in pieces: while one piece is being
// computed, the next one is on its way in over PCIe and the previous result is on its way out.
// Three streams (copy in, compute, copy out) and one event pair per piece do the ordering;
// every piece is computed by the same entry points a device-resident caller uses, on strided
// views of whole-size device buffers carved out of the caller's workspace.  The permutation is
// drawn once per call and shared by all pieces.
#include <mutex>

#include "sa_common.cuh"

namespace sa {
namespace {

constexpr int kMaxPieces = 256;

struct Piece { int ka, kb, qa, qb, with_kv; };

// KV heads in at most n_groups contiguous ranges.  The first and the last range, when they hold
// one KV head, are cut further into q_parts ranges of query heads if those divide evenly (only
// the first part carries K/V): the copy in of the first piece and the kernels and copy out of
// the last one are what cannot overlap, so those pieces are small; the pieces in between are
// large, because every piece costs launches and events.
int plan(int Hq, int Hkv, int n_groups, int q_parts, Piece* out, int max_out) {
  if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || !out) return -1;
  const int G = Hq / Hkv;
  n_groups = n_groups < 1 ? 1 : (n_groups > Hkv ? Hkv : n_groups);
  int cnt = 0;
  for (int i = 0; i < n_groups; ++i) {
    const int a = (int)((int64_t)i * Hkv / n_groups), b = (int)((int64_t)(i + 1) * Hkv / n_groups);
    if (b <= a) continue;
    const bool edge = i == 0 || i == n_groups - 1;
    if (edge && b - a == 1 && q_parts > 1 && G % q_parts == 0) {
      const int step = G / q_parts;
      for (int j = 0; j < q_parts; ++j) {
        if (cnt >= max_out) return -1;
        out[cnt++] = Piece{a, b, a * G + j * step, a * G + (j + 1) * step, j == 0};
      }
    } else {
      if (cnt >= max_out) return -1;
      out[cnt++] = Piece{a, b, a * G, b * G, 1};
    }
  }
  return cnt;
}

// Streams and events of the pipeline, created at the first call on a device and kept.
struct Pipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_end = nullptr;
  cudaEvent_t ev_in[kMaxPieces], ev_done[kMaxPieces];
};
Pipe g_pipes[64];
std::mutex g_pipe_mutex;

Pipe* pipe_for_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  Pipe& p = g_pipes[dev];
  if (p.ready) return &p;
  bool ok = cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p.s_run, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.ev_start, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.ev_end, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < kMaxPieces; ++i)
    ok = cudaEventCreateWithFlags(&p.ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&p.ev_done[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) return nullptr;
  p.ready = true;
  return &p;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct Carve {
  size_t q, k, v, y, scratch, gate, perm, inv, perm_ws, total;
};

bool carve(const sa_problem* p, Carve* c) {
  if (!p || p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->n < 1 || p->d < 1) return false;
  const size_t es = p->dtype == SA_BF16 ? 2 : 4;
  const size_t qb = (size_t)p->B * p->Hq * p->n * p->d * es;
  const size_t kb = (size_t)p->B * p->Hkv * p->n * p->d * es;
  size_t o = 0;
  c->q = o; o += align256(qb);
  c->k = o; o += align256(kb);
  c->v = o; o += align256(kb);
  c->y = o; o += align256(qb);
  c->scratch = o; o += align256(qb);
  // the logits as they come ([2, Hq]), then one contiguous [2, heads] block per piece
  c->gate = o; o += 2 * align256((size_t)2 * p->Hq * sizeof(float));
  c->perm = o; o += align256((size_t)p->B * p->n * sizeof(int32_t));
  c->inv = o; o += align256((size_t)p->B * p->n * sizeof(int32_t));
  c->perm_ws = o; o += align256(make_perm_ws_bytes(p->B, p->n));
  c->total = o;
  return true;
}

}  // namespace
}  // namespace sa

using namespace sa;

extern "C" {

int32_t sa_host_forward_plan(int32_t Hq, int32_t Hkv, int32_t n_groups, int32_t q_parts,
                             int32_t* pieces, int32_t max_pieces) {
  Piece tmp[kMaxPieces];
  const int cnt = plan(Hq, Hkv, n_groups, q_parts, tmp, kMaxPieces);
  if (cnt < 0 || cnt > max_pieces || !pieces) return -1;
  for (int i = 0; i < cnt; ++i) {
    pieces[5 * i + 0] = tmp[i].ka; pieces[5 * i + 1] = tmp[i].kb;
    pieces[5 * i + 2] = tmp[i].qa; pieces[5 * i + 3] = tmp[i].qb;
    pieces[5 * i + 4] = tmp[i].with_kv;
  }
  return cnt;
}

size_t sa_host_forward_ws_bytes(const sa_problem* p) {
  Carve c;
  return carve(p, &c) ? c.total : (size_t)-1;
}

sa_status sa_swa_gated_forward_host(const sa_problem* p, const void* q, const void* k,
                                    const void* v, const float* gate_logits, void* y,
                                    uint64_t seed, uint32_t layer, int32_t n_groups,
                                    int32_t q_parts, void* ws, size_t ws_bytes,
                                    sa_stream_t stream) {
  if (!p || !q || !k || !v || !gate_logits || !y || !ws) return SA_ERR_INVALID_ARG;
  if (((uintptr_t)ws & 255u) != 0) return SA_ERR_INVALID_ARG;
  Carve c;
  if (!carve(p, &c)) return SA_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return SA_ERR_WORKSPACE;
  Piece pieces[kMaxPieces];
  const int cnt = plan(p->Hq, p->Hkv, n_groups, q_parts, pieces, kMaxPieces);
  if (cnt < 1) return SA_ERR_INVALID_ARG;
  // device-side problem: contiguous [B,H,n,d] buffers, whatever the strides field says
  sa_problem dp = *p;
  sa_problem_set_contiguous(&dp);
  dp.flags &= ~(uint32_t)SA_SAVE_FOR_BWD;
  // validate the shape once through the ordinary sizing call
  if (sa_workspace_bytes(&dp, SA_OP_GATED_FORWARD) == (size_t)-1) return SA_ERR_INVALID_ARG;
  Pipe* pipe = pipe_for_current_device();
  if (!pipe) return SA_ERR_CUDA;

  char* base = (char*)ws;
  const size_t es = p->dtype == SA_BF16 ? 2 : 4;
  const size_t head_bytes = (size_t)p->n * p->d * es;
  char *dq = base + c.q, *dk = base + c.k, *dv = base + c.v, *dyv = base + c.y;
  float* dgate_all = (float*)(base + c.gate);
  float* dgate = (float*)(base + c.gate + align256((size_t)2 * p->Hq * sizeof(float)));
  int32_t* dperm = (int32_t*)(base + c.perm);
  int32_t* dinv = (int32_t*)(base + c.inv);
  cudaStream_t cur = (cudaStream_t)stream;
  bool ok = true;
  auto chk = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };

  // everything below is ordered after what the caller's stream has queued so far
  chk(cudaEventRecord(pipe->ev_start, cur));
  chk(cudaStreamWaitEvent(pipe->s_in, pipe->ev_start, 0));
  chk(cudaStreamWaitEvent(pipe->s_run, pipe->ev_start, 0));
  chk(cudaStreamWaitEvent(pipe->s_out, pipe->ev_start, 0));

  // copy in: all logits in one small copy (a copy of a few bytes holds the copy engine as long
  // as one of a few hundred kilobytes, and two per piece stood between the large ones), then
  // the heads of each piece; the [2, heads] block of a piece is cut out on the compute stream
  chk(cudaMemcpyAsync(dgate_all, gate_logits, (size_t)2 * p->Hq * sizeof(float),
                      cudaMemcpyHostToDevice, pipe->s_in));
  size_t gate_off = 0;
  size_t gate_at[kMaxPieces];
  for (int i = 0; i < cnt && ok; ++i) {
    const Piece& g = pieces[i];
    const int hq = g.qb - g.qa;
    gate_at[i] = gate_off;
    gate_off += (size_t)2 * hq;
    for (int b = 0; b < p->B; ++b) {   // one contiguous block per sequence and tensor
      if (g.with_kv) {
        const size_t off = ((size_t)b * p->Hkv + g.ka) * head_bytes, len = (size_t)(g.kb - g.ka) * head_bytes;
        chk(cudaMemcpyAsync(dk + off, (const char*)k + off, len, cudaMemcpyHostToDevice, pipe->s_in));
        chk(cudaMemcpyAsync(dv + off, (const char*)v + off, len, cudaMemcpyHostToDevice, pipe->s_in));
      }
      const size_t off = ((size_t)b * p->Hq + g.qa) * head_bytes, len = (size_t)hq * head_bytes;
      chk(cudaMemcpyAsync(dq + off, (const char*)q + off, len, cudaMemcpyHostToDevice, pipe->s_in));
    }
    chk(cudaEventRecord(pipe->ev_in[i], pipe->s_in));
  }

  // compute: fresh permutation, then piece by piece as the inputs arrive
  sa_status st = SA_OK;
  if (ok)
    st = sa_make_perm(seed, layer, p->B, p->n, dperm, dinv, base + c.perm_ws,
                      make_perm_ws_bytes(p->B, p->n), (sa_stream_t)pipe->s_run);
  for (int i = 0; i < cnt && ok && st == SA_OK; ++i) {
    const Piece& g = pieces[i];
    chk(cudaStreamWaitEvent(pipe->s_run, pipe->ev_in[i], 0));
    chk(cudaMemcpy2DAsync(dgate + gate_at[i], (size_t)(g.qb - g.qa) * sizeof(float), dgate_all + g.qa,
                          (size_t)p->Hq * sizeof(float), (size_t)(g.qb - g.qa) * sizeof(float), 2,
                          cudaMemcpyDeviceToDevice, pipe->s_run));
    sa_problem gp = dp;                     // a view of the whole-size buffers: same strides
    gp.Hq = g.qb - g.qa;
    gp.Hkv = g.kb - g.ka;
    const size_t qoff = (size_t)g.qa * head_bytes, koff = (size_t)g.ka * head_bytes;
    st = sa_swa_gated_forward(&gp, dq + qoff, dk + koff, dv + koff, dperm, dinv,
                              dgate + gate_at[i], dyv + qoff, nullptr, nullptr, nullptr, nullptr,
                              base + c.scratch, (size_t)(c.gate - c.scratch),
                              (sa_stream_t)pipe->s_run);
    chk(cudaEventRecord(pipe->ev_done[i], pipe->s_run));
  }

  // copy out
  for (int i = 0; i < cnt && ok && st == SA_OK; ++i) {
    const Piece& g = pieces[i];
    chk(cudaStreamWaitEvent(pipe->s_out, pipe->ev_done[i], 0));
    for (int b = 0; b < p->B; ++b) {
      const size_t off = ((size_t)b * p->Hq + g.qa) * head_bytes, len = (size_t)(g.qb - g.qa) * head_bytes;
      chk(cudaMemcpyAsync((char*)y + off, dyv + off, len, cudaMemcpyDeviceToHost, pipe->s_out));
    }
  }
  // the caller's stream resumes when all three streams are done (also after an error, so
  // that nothing of this call is still in flight when the caller goes on)
  cudaEventRecord(pipe->ev_end, pipe->s_in);
  cudaStreamWaitEvent(cur, pipe->ev_end, 0);
  cudaEventRecord(pipe->ev_end, pipe->s_run);
  cudaStreamWaitEvent(cur, pipe->ev_end, 0);
  cudaEventRecord(pipe->ev_end, pipe->s_out);
  cudaStreamWaitEvent(cur, pipe->ev_end, 0);
  if (st != SA_OK) return st;
  return ok ? SA_OK : SA_ERR_CUDA;
}

}  // extern "C"
