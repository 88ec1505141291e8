// C-ABI entry points of the SwiLA library: host-side validation and kernel dispatch.
// No device memory is allocated here; the only host-side state kept between calls is the pair of copy streams (and
// their events) that the host-buffer front end creates per device on first use for problems of 64 MB and more.  (The
// library image itself carries three device arrays: the staging array of the allocation-free entry point, and the
// hand-over flags and the error word of the chunked kernel.)
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "../../include/swila_dev.h"
#include "swila_common.cuh"

namespace swila {
#define SWILA_DECL(DK, GATE, POST) template <> int scan_dispatch<DK, GATE, POST>(const LaunchArgs &);
#define SWILA_DECL_DK(DK) \
  SWILA_DECL(DK, 0, false) SWILA_DECL(DK, 1, false) SWILA_DECL(DK, 1, true) SWILA_DECL(DK, 2, false) SWILA_DECL(DK, 2, true) \
      SWILA_DECL(DK, 3, false) SWILA_DECL(DK, 3, true)
SWILA_DECL_DK(16)
SWILA_DECL_DK(64)
SWILA_DECL_DK(128)

int chunk_dispatch(const LaunchArgs &a);
int chunk_gated_dispatch(LaunchArgs &a);
int chunk_error_fetch(int *flag);
int chunk_gated_error_fetch(int *flag);

static thread_local char g_cuda_err[256] = "";

static int cuda_fail(cudaError_t e) {
  strncpy(g_cuda_err, cudaGetErrorString(e), sizeof(g_cuda_err) - 1);
  g_cuda_err[sizeof(g_cuda_err) - 1] = 0;
  return SWILA_ERR_CUDA;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_shape(const swila_shape_t *s, bool need_T) {
  if (!s) return SWILA_ERR_NULL;
  if (s->B <= 0 || s->H <= 0 || s->Dk <= 0 || s->Dv <= 0 || s->J <= 0) return SWILA_ERR_SHAPE;
  if (need_T && s->T < 0) return SWILA_ERR_SHAPE;
  if (s->Dv % 8 != 0) return SWILA_ERR_SHAPE;
  if (s->Dk != 16 && s->Dk != 64 && s->Dk != 128) return SWILA_ERR_UNSUPPORTED;
  if (s->J != 1 && s->J != 2 && s->J != 4 && s->J != 8 && s->J != 16) return SWILA_ERR_UNSUPPORTED;
  if (s->io_dtype != SWILA_IO_FP32 && s->io_dtype != SWILA_IO_BF16) return SWILA_ERR_UNSUPPORTED;
  if (s->flags & ~(SWILA_TEMPORAL | SWILA_GATED | SWILA_POST_DECAY | SWILA_QKV_ACT)) return SWILA_ERR_UNSUPPORTED;
  const bool gated = (s->flags & SWILA_GATED) != 0;
  if (!gated && (s->flags & SWILA_POST_DECAY)) return SWILA_ERR_UNSUPPORTED;
  if (gated != (s->gate_granularity != SWILA_GATE_NONE)) return SWILA_ERR_UNSUPPORTED;
  if (s->gate_granularity < SWILA_GATE_NONE || s->gate_granularity > SWILA_GATE_ELEMENTWISE) return SWILA_ERR_UNSUPPORTED;
  if (s->algo != SWILA_ALGO_AUTO && s->algo != SWILA_ALGO_SCAN && s->algo != SWILA_ALGO_SCAN_WIDE &&
      s->algo != SWILA_ALGO_SCAN_NARROW && s->algo != SWILA_ALGO_CHUNK)
    return SWILA_ERR_UNSUPPORTED;
  return SWILA_OK;
}

static size_t w_elems(const swila_shape_t *s) { return (size_t)s->B * s->H * s->J * s->Dv * s->Dk; }
static size_t r_elems(const swila_shape_t *s) { return (size_t)s->B * s->H * s->J * s->Dv; }

// elements of alpha for T tokens, by granularity
static size_t alpha_elems(const swila_shape_t *s, int T) {
  const size_t ntok = (size_t)s->B * s->H * (size_t)T;
  switch (s->gate_granularity) {
    case SWILA_GATE_PER_KEY: return ntok * s->J * s->Dk;
    case SWILA_GATE_PER_OUT: return ntok * s->J * s->Dv;
    case SWILA_GATE_SCALAR: return ntok * s->J;
    case SWILA_GATE_ELEMENTWISE: return ntok * s->J * s->Dv * s->Dk;
    default: return 0;
  }
}

static bool overlaps(const void *a, size_t na, const void *b, size_t nb) {
  if (!a || !b || na == 0 || nb == 0) return false;
  const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
  return a0 < b0 + nb && b0 < a0 + na;
}

// What the chunked tensor-core kernel covers (the AUTO rule of swila_forward is this and T >= 64): bf16 io, Dk in
// {64, 128}, J in {4, 8} or J = 16 at Dk = 64, plain or Temporal, or Gated with one decay per state row; auxiliary
// outputs (r_debug, statistics) for the ungated shapes with J <= 8.
static bool chunk_covers(const swila_shape_t *s, bool aux) {
  if (s->io_dtype != SWILA_IO_BF16 || (s->Dk != 64 && s->Dk != 128)) return false;
  if (s->flags & SWILA_QKV_ACT) return false;
  if (s->flags & SWILA_GATED) {  // one decay per state row (per output dimension, or per component), pre- or post-decay
    if (s->gate_granularity != SWILA_GATE_PER_OUT && s->gate_granularity != SWILA_GATE_SCALAR) return false;
    if ((s->flags & SWILA_TEMPORAL) && s->Dk != 64) return false;
    return (s->J == 4 || (s->J == 8 && s->Dk == 64)) && !aux;
  }
  if (!(s->J == 4 || s->J == 8 || (s->J == 16 && s->Dk == 64))) return false;
  if (aux && s->J == 16) return false;
  return true;
}

static int run(const swila_shape_t *s, int T, const void *q, const void *k, const void *v, const swila_gates_t *g,
               const swila_state_t *sin, swila_state_t *sout, void *o, float *r_debug, void *stream,
               const swila_stats_t *stats = nullptr) {
  const bool temporal = (s->flags & SWILA_TEMPORAL) != 0;
  const bool gated = (s->flags & SWILA_GATED) != 0;
  if (!q || !k || !v || !g || !o) return SWILA_ERR_NULL;
  if (!g->beta_logit || !g->pik_logit || !g->piq_logit) return SWILA_ERR_NULL;
  if (temporal && (!g->gk_logit || !g->gq_logit)) return SWILA_ERR_NULL;
  if (gated && !g->alpha) return SWILA_ERR_NULL;
  if (sin && !sin->W) return SWILA_ERR_NULL;
  if (sout && !sout->W) return SWILA_ERR_NULL;
  if (temporal && sin && (!sin->r_prev || !sin->rho_prev)) return SWILA_ERR_NULL;
  if (temporal && sout && (!sout->r_prev || !sout->rho_prev)) return SWILA_ERR_NULL;
  const void *ptrs[] = {q, k, v, o, g->beta_logit, g->pik_logit, g->piq_logit, temporal ? g->gk_logit : nullptr,
                        temporal ? g->gq_logit : nullptr, gated ? (const void *)g->alpha : nullptr,
                        sin ? sin->W : nullptr, sout ? sout->W : nullptr, r_debug};
  for (const void *p : ptrs)
    if (p && !aligned16(p)) return SWILA_ERR_ALIGN;
  const size_t es = s->io_dtype == SWILA_IO_BF16 ? 2 : 4;
  const size_t ntok = (size_t)s->B * s->H * (size_t)T;
  const size_t o_bytes = ntok * s->Dv * es;
  const size_t gate_bytes = ntok * s->J * s->Dv * es;
  {
    // Both kernels read the streamed inputs ahead of the tokens they write (cp.async ring, tensor copies), so
    // nothing that is written may overlap them; the written tensors must not overlap one another either.
    struct Range { const void *p; size_t n; };
    const Range in[] = {{q, ntok * s->Dk * es}, {k, ntok * s->Dk * es}, {v, ntok * s->Dv * es},
                        {g->beta_logit, gate_bytes}, {g->pik_logit, gate_bytes}, {g->piq_logit, gate_bytes},
                        {temporal ? g->gk_logit : nullptr, ntok * s->Dv * es},
                        {temporal ? g->gq_logit : nullptr, ntok * s->Dv * es},
                        {gated ? (const void *)g->alpha : nullptr, alpha_elems(s, T) * 4}};
    const Range out[] = {{o, o_bytes}, {r_debug, ntok * s->J * s->Dv * 4},
                         {sout ? sout->W : nullptr, w_elems(s) * 4},
                         {(sout && temporal) ? sout->r_prev : nullptr, r_elems(s) * 4},
                         {(sout && temporal) ? sout->rho_prev : nullptr, r_elems(s) * 4}};
    for (const Range &w : out)
      for (const Range &r : in)
        if (overlaps(w.p, w.n, r.p, r.n)) return SWILA_ERR_ALIAS;
    for (size_t i = 0; i < sizeof(out) / sizeof(out[0]); ++i)
      for (size_t j = i + 1; j < sizeof(out) / sizeof(out[0]); ++j)
        if (overlaps(out[i].p, out[i].n, out[j].p, out[j].n)) return SWILA_ERR_ALIAS;
    if (sin) {  // the initial state may be the output state itself (in place), nothing else that is written
      const Range st[] = {{sin->W, w_elems(s) * 4}, {temporal ? sin->r_prev : nullptr, r_elems(s) * 4},
                          {temporal ? sin->rho_prev : nullptr, r_elems(s) * 4}};
      for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 5; ++j)
          if (!(j == 2 + i && st[i].p == out[j].p) && overlaps(st[i].p, st[i].n, out[j].p, out[j].n)) return SWILA_ERR_ALIAS;
    }
  }

  LaunchArgs a;
  memset(&a, 0, sizeof(a));
  a.p.B = s->B; a.p.H = s->H; a.p.T = T; a.p.Dv = s->Dv;
  a.p.temporal = temporal ? 1 : 0;
  a.p.gran = s->gate_granularity;
  a.p.q = q; a.p.k = k; a.p.v = v;
  a.p.beta_logit = g->beta_logit; a.p.pik_logit = g->pik_logit; a.p.piq_logit = g->piq_logit;
  a.p.gk_logit = temporal ? g->gk_logit : nullptr;
  a.p.gq_logit = temporal ? g->gq_logit : nullptr;
  a.p.alpha = gated ? g->alpha : nullptr;
  a.p.W_in = sin ? sin->W : nullptr;
  a.p.r_in = (sin && temporal) ? sin->r_prev : nullptr;
  a.p.rho_in = (sin && temporal) ? sin->rho_prev : nullptr;
  a.p.W_out = sout ? sout->W : nullptr;
  a.p.r_out = (sout && temporal) ? sout->r_prev : nullptr;
  a.p.rho_out = (sout && temporal) ? sout->rho_prev : nullptr;
  a.p.o = o;
  a.p.r_debug = r_debug;
  a.p.qkv_act = (s->flags & SWILA_QKV_ACT) ? 1 : 0;
  a.p.post = (s->flags & SWILA_POST_DECAY) ? 1 : 0;
  if (stats) {
    a.p.r_sum = stats->r_sum; a.p.r_ent = stats->r_ent;
    a.p.rho_sum = stats->rho_sum; a.p.rho_ent = stats->rho_ent;
  }
  a.Dk = s->Dk; a.J = s->J; a.io_dtype = s->io_dtype;
  a.gate_mode = !gated ? 0 : (s->gate_granularity == SWILA_GATE_PER_KEY ? 1 : s->gate_granularity == SWILA_GATE_ELEMENTWISE ? 3 : 2);
  a.post = (s->flags & SWILA_POST_DECAY) ? 1 : 0;
  a.algo = s->algo;
  a.stream = (cudaStream_t)stream;

  int rc = -1000;
  const bool aux = r_debug || a.p.r_sum || a.p.r_ent || a.p.rho_sum || a.p.rho_ent;
  const bool chunk_ok = chunk_covers(s, aux);
  if (s->algo == SWILA_ALGO_CHUNK || (s->algo == SWILA_ALGO_AUTO && chunk_ok && T >= 64)) {
    const bool gated_rows = gated && a.gate_mode == 2;
    rc = gated_rows ? chunk_gated_dispatch(a) : chunk_dispatch(a);
    if (rc == -1000 && s->algo == SWILA_ALGO_CHUNK) return SWILA_ERR_UNSUPPORTED;
    if (rc != -1000) {
      if (rc != 0) return cuda_fail((cudaError_t)rc);
      if (!gated_rows) return SWILA_OK;
      // Gated rows: the scan kernel is launched behind the chunked one; exactly one of the two does the work,
      // as the guard pass over the decays has decided (chunk_gated_dispatch)
      a.p.guard_runs_scan = 1;
      a.algo = SWILA_ALGO_SCAN;
    }
  }
#define SWILA_CASE(DK)                                                                          \
  case DK:                                                                                      \
    if (a.gate_mode == 0) rc = scan_dispatch<DK, 0, false>(a);                                  \
    else if (a.gate_mode == 1) rc = a.post ? scan_dispatch<DK, 1, true>(a) : scan_dispatch<DK, 1, false>(a); \
    else if (a.gate_mode == 3) rc = a.post ? scan_dispatch<DK, 3, true>(a) : scan_dispatch<DK, 3, false>(a); \
    else rc = a.post ? scan_dispatch<DK, 2, true>(a) : scan_dispatch<DK, 2, false>(a);          \
    break;
  switch (s->Dk) {
    SWILA_CASE(16)
    SWILA_CASE(64)
    SWILA_CASE(128)
    default: break;
  }
  if (rc == -1000) return SWILA_ERR_UNSUPPORTED;
  if (rc != 0) return cuda_fail((cudaError_t)rc);
  return SWILA_OK;
}

__global__ void fill_kernel(float *p, size_t n, float val) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) p[i] = val;
}

}  // namespace swila

using namespace swila;

extern "C" {

int swila_version(void) { return 200; }

int swila_auto_algo(const swila_shape_t *s, int aux_outputs) {
  int rc = check_shape(s, true);
  if (rc) return rc;
  return (chunk_covers(s, aux_outputs != 0) && s->T >= 64) ? SWILA_ALGO_CHUNK : SWILA_ALGO_SCAN;
}

const char *swila_strerror(int status) {
  switch (status) {
    case SWILA_OK: return "ok";
    case SWILA_ERR_NULL: return "a required pointer is NULL";
    case SWILA_ERR_SHAPE: return "invalid shape (non-positive dimension, or Dv not a multiple of 8)";
    case SWILA_ERR_UNSUPPORTED: return "unsupported Dk / J / dtype / flag combination";
    case SWILA_ERR_ALIGN: return "a pointer is not 16-byte aligned";
    case SWILA_ERR_ALIAS: return "the output overlaps an input";
    case SWILA_ERR_CUDA: return "a CUDA runtime call failed (see swila_last_cuda_error)";
    case SWILA_ERR_SIZE: return "problem exceeds a size limit of this entry point";
    default: return "unknown status";
  }
}

const char *swila_last_cuda_error(void) { return g_cuda_err; }

int swila_device_status(void) {
  int flag = 0;
  cudaError_t e = (cudaError_t)chunk_error_fetch(&flag);  // (the error word exists once per translation unit)
  if (e != cudaSuccess) return cuda_fail(e);
  if (!flag) {
    e = (cudaError_t)chunk_gated_error_fetch(&flag);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (flag) {  // (warp + 1) << 16 | low half of the barrier's shared-memory address; 1 if only a hand-over flag gave up
    snprintf(g_cuda_err, sizeof(g_cuda_err), "a bounded wait expired inside the chunked kernel (warp %d, barrier at 0x%x)",
             (flag >> 16) - 1, flag & 0xffff);
    return SWILA_ERR_CUDA;
  }
  return SWILA_OK;
}

size_t swila_state_w_bytes(const swila_shape_t *s) { return check_shape(s, false) == SWILA_OK ? w_elems(s) * 4 : 0; }
size_t swila_state_r_bytes(const swila_shape_t *s) { return check_shape(s, false) == SWILA_OK ? r_elems(s) * 4 : 0; }

int swila_state_init(const swila_shape_t *s, swila_state_t *st, void *stream) {
  int rc = check_shape(s, false);
  if (rc) return rc;
  if (!st || !st->W) return SWILA_ERR_NULL;
  const bool temporal = (s->flags & SWILA_TEMPORAL) != 0;
  if (temporal && (!st->r_prev || !st->rho_prev)) return SWILA_ERR_NULL;
  cudaStream_t cs = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(st->W, 0, w_elems(s) * 4, cs);
  if (e != cudaSuccess) return cuda_fail(e);
  if (temporal) {
    const size_t n = r_elems(s);
    const unsigned grid = (unsigned)((n + 255) / 256 < 1024 ? (n + 255) / 256 : 1024);
    fill_kernel<<<grid, 256, 0, cs>>>(st->r_prev, n, 1.0f / s->J);
    fill_kernel<<<grid, 256, 0, cs>>>(st->rho_prev, n, 1.0f / s->J);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return SWILA_OK;
}

int swila_forward(const swila_shape_t *s, const void *q, const void *k, const void *v, const swila_gates_t *g,
                  const swila_state_t *state_in, swila_state_t *state_out, void *o, float *r_debug, void *stream) {
  int rc = check_shape(s, true);
  if (rc) return rc;
  if (s->T == 0) {  // nothing to scan: the state passes through
    if (!state_out) return SWILA_OK;
    if (!state_out->W) return SWILA_ERR_NULL;
    const bool temporal = (s->flags & SWILA_TEMPORAL) != 0;
    if (temporal && (!state_out->r_prev || !state_out->rho_prev)) return SWILA_ERR_NULL;
    if (!state_in) return swila_state_init(s, state_out, stream);
    if (!state_in->W || (temporal && (!state_in->r_prev || !state_in->rho_prev))) return SWILA_ERR_NULL;
    cudaStream_t cs = (cudaStream_t)stream;
    cudaError_t e = cudaSuccess;
    if (state_in->W != state_out->W)
      e = cudaMemcpyAsync(state_out->W, state_in->W, w_elems(s) * 4, cudaMemcpyDeviceToDevice, cs);
    if (e == cudaSuccess && temporal && state_in->r_prev != state_out->r_prev)
      e = cudaMemcpyAsync(state_out->r_prev, state_in->r_prev, r_elems(s) * 4, cudaMemcpyDeviceToDevice, cs);
    if (e == cudaSuccess && temporal && state_in->rho_prev != state_out->rho_prev)
      e = cudaMemcpyAsync(state_out->rho_prev, state_in->rho_prev, r_elems(s) * 4, cudaMemcpyDeviceToDevice, cs);
    return e == cudaSuccess ? SWILA_OK : cuda_fail(e);
  }
  return run(s, s->T, q, k, v, g, state_in, state_out, o, r_debug, stream);
}

int swila_forward_stats(const swila_shape_t *s, const void *q, const void *k, const void *v, const swila_gates_t *g,
                        const swila_state_t *state_in, swila_state_t *state_out, void *o, float *r_debug,
                        const swila_stats_t *stats, void *stream) {
  int rc = check_shape(s, true);
  if (rc) return rc;
  if (!stats) return SWILA_ERR_NULL;
  if (s->T == 0) return swila_forward(s, q, k, v, g, state_in, state_out, o, r_debug, stream);  // nothing to add
  return run(s, s->T, q, k, v, g, state_in, state_out, o, r_debug, stream, stats);
}

int swila_decode_step(const swila_shape_t *s, const void *q, const void *k, const void *v, const swila_gates_t *g,
                      swila_state_t *state, void *o, void *stream) {
  int rc = check_shape(s, false);
  if (rc) return rc;
  if (!state) return SWILA_ERR_NULL;
  swila_shape_t one = *s;  // a single token always goes through the scan kernel (bit-equal to a scan prefill)
  if (one.algo == SWILA_ALGO_CHUNK) one.algo = SWILA_ALGO_SCAN;
  return run(&one, 1, q, k, v, g, state, state, o, nullptr, stream);
}

}  // extern "C"

// ---- host-buffer front end --------------------------------------------------------------
namespace swila {
static size_t up256(size_t n) { return (n + 255) & ~(size_t)255; }
struct HostPlan {
  size_t q, k, v, beta, pik, piq, gk, gq, alpha, W, r, rho, o, total;
  size_t n_qk, n_v, n_gate, n_tg, n_alpha, n_W, n_r;
};
static HostPlan host_plan(const swila_shape_t *s) {
  HostPlan h;
  const size_t es = s->io_dtype == SWILA_IO_BF16 ? 2 : 4;
  const size_t ntok = (size_t)s->B * s->H * (size_t)s->T;
  const bool temporal = (s->flags & SWILA_TEMPORAL) != 0, gated = (s->flags & SWILA_GATED) != 0;
  h.n_qk = ntok * s->Dk * es;
  h.n_v = ntok * s->Dv * es;
  h.n_gate = ntok * s->J * s->Dv * es;
  h.n_tg = temporal ? ntok * s->Dv * es : 0;
  h.n_alpha = gated ? alpha_elems(s, s->T) * 4 : 0;
  h.n_W = w_elems(s) * 4;
  h.n_r = temporal ? r_elems(s) * 4 : 0;
  size_t off = 0;
  auto take = [&](size_t n) { size_t o = off; off += up256(n); return o; };
  h.q = take(h.n_qk); h.k = take(h.n_qk); h.v = take(h.n_v);
  h.beta = take(h.n_gate); h.pik = take(h.n_gate); h.piq = take(h.n_gate);
  h.gk = take(h.n_tg); h.gq = take(h.n_tg); h.alpha = take(h.n_alpha);
  h.W = take(h.n_W); h.r = take(h.n_r); h.rho = take(h.n_r);
  h.o = take(h.n_v);
  h.total = off;
  return h;
}
}  // namespace swila

extern "C" {

size_t swila_forward_host_workspace_bytes(const swila_shape_t *s) {
  if (check_shape(s, true) != SWILA_OK) return 0;
  return host_plan(s).total;
}

}  // extern "C"

// Streams and events of the pipelined host path, one set per device, created on first use and kept.
namespace swila {
constexpr int kHostSlabs = 8;
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done = nullptr, landed[kHostSlabs] = {}, computed[kHostSlabs] = {};
  // Held by a call for its whole enqueue phase: every event above is recorded on one stream and waited for on
  // another, and a wait refers to the latest record at the time it is enqueued, so the record/wait pairs of two
  // host threads must not interleave.  (Their GPU work may: each call has its own workspace.)
  std::mutex enqueue;
};
static HostPipe *host_pipe() {
  static std::mutex mu;
  static HostPipe pipes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe &hp = pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kHostSlabs; ++i)
      ok = cudaEventCreateWithFlags(&hp.landed[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      (void)cudaGetLastError();
      return nullptr;
    }
    hp.ready = true;
  }
  return &hp;
}
}  // namespace swila

extern "C" {

int swila_forward_host(const swila_shape_t *s, const void *q, const void *k, const void *v, const swila_gates_t *g,
                       const swila_state_t *state_in, swila_state_t *state_out, void *o, void *workspace,
                       size_t workspace_bytes, void *stream) {
  int rc = check_shape(s, true);
  if (rc) return rc;
  if (!q || !k || !v || !g || !o || !workspace) return SWILA_ERR_NULL;
  const bool temporal = (s->flags & SWILA_TEMPORAL) != 0, gated = (s->flags & SWILA_GATED) != 0;
  if (!g->beta_logit || !g->pik_logit || !g->piq_logit) return SWILA_ERR_NULL;
  if (temporal && (!g->gk_logit || !g->gq_logit)) return SWILA_ERR_NULL;
  if (gated && !g->alpha) return SWILA_ERR_NULL;
  if (state_in && (!state_in->W || (temporal && (!state_in->r_prev || !state_in->rho_prev)))) return SWILA_ERR_NULL;
  if (state_out && (!state_out->W || (temporal && (!state_out->r_prev || !state_out->rho_prev)))) return SWILA_ERR_NULL;
  if (!aligned16(workspace)) return SWILA_ERR_ALIGN;
  const HostPlan h = host_plan(s);
  if (workspace_bytes < h.total) return SWILA_ERR_SIZE;
  char *ws = (char *)workspace;
  cudaStream_t cs = (cudaStream_t)stream;
  cudaError_t e = cudaSuccess;

  // Every tensor is [B*H, ...] with the (batch, head) index outermost, and (batch, head) pairs are independent: large
  // problems go through in slabs of (batch, head) pairs, the host-to-device copies of slab i+1 and the device-to-host
  // copies of slab i-1 running on two internal streams beside the kernel of slab i on `stream`.  The call still
  // returns without synchronising and `stream` is complete when everything is (it waits for the internal streams).
  const long long nbh = (long long)s->B * s->H;
  auto slab_ok = [&](size_t total) { return (total / (size_t)nbh) % 16 == 0; };  // slab bases stay 16-byte aligned
  const bool sliceable = slab_ok(h.n_qk) && slab_ok(h.n_v) && slab_ok(h.n_gate) && slab_ok(h.n_tg) && slab_ok(h.n_alpha) &&
                         slab_ok(h.n_W) && slab_ok(h.n_r);
  HostPipe *hp = (h.total >= (64u << 20) && nbh >= 2 && sliceable) ? host_pipe() : nullptr;
  const int nslab = hp ? (int)(nbh < kHostSlabs ? nbh : kHostSlabs) : 1;
  cudaStream_t s_in = hp ? hp->in : cs, s_out = hp ? hp->out : cs;
  std::unique_lock<std::mutex> enqueue_lock;
  if (hp) enqueue_lock = std::unique_lock<std::mutex>(hp->enqueue);
  if (hp) {
    e = cudaEventRecord(hp->start, cs);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s_in, hp->start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, hp->start, 0);
  }
  swila_shape_t sub = *s;
  sub.B = 1;
  for (int i = 0; i < nslab && e == cudaSuccess; ++i) {
    const long long bh0 = nbh * i / nslab, bh1 = nbh * (i + 1) / nslab, cnt = bh1 - bh0;
    if (cnt == 0) continue;
    sub.H = (int32_t)cnt;
    // byte range of this slab inside a tensor of `total` bytes
    auto lo = [&](size_t total) { return (size_t)(total / (size_t)nbh) * (size_t)bh0; };
    auto len = [&](size_t total) { return (size_t)(total / (size_t)nbh) * (size_t)cnt; };
    auto up = [&](size_t off, const void *src, size_t total) {
      if (e == cudaSuccess && total)
        e = cudaMemcpyAsync(ws + off + lo(total), (const char *)src + lo(total), len(total), cudaMemcpyHostToDevice, s_in);
    };
    up(h.q, q, h.n_qk); up(h.k, k, h.n_qk); up(h.v, v, h.n_v);
    up(h.beta, g->beta_logit, h.n_gate); up(h.pik, g->pik_logit, h.n_gate); up(h.piq, g->piq_logit, h.n_gate);
    if (temporal) { up(h.gk, g->gk_logit, h.n_tg); up(h.gq, g->gq_logit, h.n_tg); }
    if (gated) up(h.alpha, g->alpha, h.n_alpha);
    if (state_in) {
      up(h.W, state_in->W, h.n_W);
      if (temporal) { up(h.r, state_in->r_prev, h.n_r); up(h.rho, state_in->rho_prev, h.n_r); }
    }
    if (e != cudaSuccess) break;
    if (hp) {
      e = cudaEventRecord(hp->landed[i], s_in);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, hp->landed[i], 0);
      if (e != cudaSuccess) break;
    }
    swila_state_t dstate = {(float *)(ws + h.W + lo(h.n_W)), temporal ? (float *)(ws + h.r + lo(h.n_r)) : nullptr,
                            temporal ? (float *)(ws + h.rho + lo(h.n_r)) : nullptr};
    swila_gates_t dg = {ws + h.beta + lo(h.n_gate), ws + h.pik + lo(h.n_gate), ws + h.piq + lo(h.n_gate),
                        temporal ? ws + h.gk + lo(h.n_tg) : nullptr, temporal ? ws + h.gq + lo(h.n_tg) : nullptr,
                        gated ? (const float *)(ws + h.alpha + lo(h.n_alpha)) : nullptr};
    rc = swila_forward(&sub, ws + h.q + lo(h.n_qk), ws + h.k + lo(h.n_qk), ws + h.v + lo(h.n_v), &dg,
                       state_in ? &dstate : nullptr, state_out ? &dstate : nullptr, ws + h.o + lo(h.n_v), nullptr, stream);
    if (rc) return rc;
    if (hp) {
      e = cudaEventRecord(hp->computed[i], cs);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, hp->computed[i], 0);
      if (e != cudaSuccess) break;
    }
    auto down = [&](void *dst, size_t off, size_t total) {
      if (e == cudaSuccess && total)
        e = cudaMemcpyAsync((char *)dst + lo(total), ws + off + lo(total), len(total), cudaMemcpyDeviceToHost, s_out);
    };
    down(o, h.o, h.n_v);
    if (state_out) {
      down(state_out->W, h.W, h.n_W);
      if (temporal) { down(state_out->r_prev, h.r, h.n_r); down(state_out->rho_prev, h.rho, h.n_r); }
    }
  }
  if (hp && e == cudaSuccess) {  // `stream` ends when the last copies have: the caller synchronises on it as before
    e = cudaEventRecord(hp->done, s_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, hp->done, 0);
    if (e == cudaSuccess) e = cudaEventRecord(hp->done, s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, hp->done, 0);
  }
  return e == cudaSuccess ? SWILA_OK : cuda_fail(e);
}

}  // extern "C"
