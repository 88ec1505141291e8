/*
 * swila.h -- C ABI of the B200 (sm_100a) Switching Linear Attention recurrence.
 *
 * The library evaluates, for every (batch b, head h), the token recurrence of the SwiLA
 * layer (Sec. 3.2): the state is J linear regressors W[j] in R^{Dv x Dk} (rows = output
 * dimensions, columns = key dimensions, App. B.4).  Per token t, for all (j, d):
 *
 *   delta = v_td - w_{t-1,jd} . k_t                               (text below Eq. 3.3)
 *   r     = softmax over j of ( log prior_jd - delta^2 / 2 )       (E-step, Eq. 3.4)
 *   w_tjd = w_{t-1,jd} + beta_tjd r delta k_t                      (M-step, Eq. 3.3)
 *   o_td  = sum_j prior^q_jd  w_tjd . q_t                          (readout, Eq. 3.5, updated state)
 *
 * beta = sigmoid(beta_logit); prior = softmax over j of pik_logit, prior^q = softmax over
 * j of piq_logit (App. B.2) -- the activations are fused into the kernels, the linear
 * projections that produce the logits are not part of this library.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer owned by the caller unless a function says HOST.
 *    The library never allocates device memory at run time and keeps no per-call state.  What it
 *    holds per device for as long as it is loaded: three file-scope device arrays (the 16 MiB
 *    staging array of swila_forward_host_static, 128 KB of hand-over flags and one error word of
 *    the chunked kernel) and, after the first pipelined swila_forward_host call on a device, two
 *    internal copy streams with their events.
 *  - All tensors are contiguous, last index fastest.  Base addresses must be 16-byte
 *    aligned.  Dv must be a multiple of 8.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 *    stream).  Inputs are never written.
 *  - Every function returning int returns SWILA_OK (0) or a negative swila_status code;
 *    nothing throws, aborts or prints.  Arguments are validated on the host before any
 *    launch.
 */
#ifndef SWILA_H_
#define SWILA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum swila_status {
  SWILA_OK = 0,
  SWILA_ERR_NULL = -1,        /* a required pointer is NULL */
  SWILA_ERR_SHAPE = -2,       /* non-positive dimension, or Dv not a multiple of 8 */
  SWILA_ERR_UNSUPPORTED = -3, /* Dk / J / dtype / flag combination not compiled */
  SWILA_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned */
  SWILA_ERR_ALIAS = -5,       /* the output o overlaps an input */
  SWILA_ERR_CUDA = -6,        /* a CUDA runtime call failed; see swila_last_cuda_error() */
  SWILA_ERR_SIZE = -7         /* a problem exceeds a stated size limit of the entry point */
};

enum { SWILA_IO_FP32 = 0, SWILA_IO_BF16 = 1 };

/* flags */
enum {
  SWILA_TEMPORAL = 1,   /* Temporal SwiLA (Sec. 3.3, App. B.3) */
  SWILA_GATED = 2,      /* Gated SwiLA, pre-decay form (Eq. 3.8) unless POST_DECAY */
  SWILA_POST_DECAY = 4, /* with GATED: post-decay form (Eq. 3.7) */
  SWILA_QKV_ACT = 8     /* q, k, v are the raw projections: the kernel applies SiLU to all three and then
                           divides q and k by sqrt(sum over Dk of squares + 1e-6), as the paper's models do
                           (App. B.2, App. D.1).  The activated values stay in FP32 (no rounding to the io
                           dtype).  Scan kernels only: with SWILA_ALGO_CHUNK -> SWILA_ERR_UNSUPPORTED */
};

/* gate_granularity (App. B.4): which indices the decay alpha depends on */
enum {
  SWILA_GATE_NONE = 0,
  SWILA_GATE_PER_KEY = 1, /* alpha [B,H,T,J,Dk]: one gate per key dimension (the LM setting, App. D.3) */
  SWILA_GATE_PER_OUT = 2, /* alpha [B,H,T,J,Dv]: one gate per output dimension (Eq. 3.7 as printed) */
  SWILA_GATE_SCALAR = 3,  /* alpha [B,H,T,J]:    one gate per component */
  SWILA_GATE_ELEMENTWISE = 4 /* alpha [B,H,T,J,Dv,Dk]: one gate per state element, the general form of App. B.4 of which
                                the other three are restrictions (J*Dv*Dk values per token: small problems only) */
};

/* algo: which kernel evaluates the recurrence.  Every choice computes the same function; what each
 * kernel covers and what AUTO picks is part of the contract of swila_forward below. */
enum {
  SWILA_ALGO_AUTO = 0,        /* the library chooses (see swila_forward) */
  SWILA_ALGO_SCAN = 1,        /* sequential scan, state resident in registers, FP32 FMA pipe; every shape */
  SWILA_ALGO_SCAN_WIDE = 2,   /* the same scan with 256-thread blocks; ungated shapes with Dk = 128 only */
  SWILA_ALGO_SCAN_NARROW = 3, /* the same scan with 16 key dimensions per lane; ungated, Dk = 128, J >= 4 only */
  SWILA_ALGO_CHUNK = 4        /* chunked form on the tcgen05 tensor cores (see swila_forward) */
};

typedef struct {
  int32_t B, H, T;          /* batch, heads, tokens (T >= 0; ignored by swila_decode_step) */
  int32_t Dk, Dv;           /* key / value head dimension; Dk in {16, 64, 128}; Dv % 8 == 0 */
  int32_t J;                /* mixture components, in {1, 2, 4, 8, 16} */
  int32_t io_dtype;         /* SWILA_IO_*: dtype of q, k, v, o and of every *_logit tensor */
  int32_t flags;            /* SWILA_TEMPORAL | SWILA_GATED | SWILA_POST_DECAY | SWILA_QKV_ACT */
  int32_t gate_granularity; /* SWILA_GATE_*; must be NONE iff GATED is clear */
  int32_t algo;             /* SWILA_ALGO_* */
} swila_shape_t;

/* Per-token gate tensors: the layer's learned projections evaluated at every token,
 * BEFORE their activation (App. B.2, B.3).  Logit tensors have the io dtype; alpha is
 * always fp32 and already in [0, 1]. */
typedef struct {
  const void *beta_logit;  /* [B,H,T,J,Dv]  beta = sigmoid(.)                        */
  const void *pik_logit;   /* [B,H,T,J,Dv]  key-side prior  = softmax over J         */
  const void *piq_logit;   /* [B,H,T,J,Dv]  query-side prior = softmax over J        */
  const void *gk_logit;    /* [B,H,T,Dv]    TEMPORAL only: g^k = sigmoid(.), else NULL */
  const void *gq_logit;    /* [B,H,T,Dv]    TEMPORAL only: g^q = sigmoid(.), else NULL */
  const float *alpha;      /* GATED only: decay, shape by gate_granularity, else NULL */
} swila_gates_t;

/* Carried state, always fp32. */
typedef struct {
  float *W;         /* [B,H,J,Dv,Dk] */
  float *r_prev;    /* [B,H,J,Dv]  TEMPORAL only: previous posterior r_{t-1}   (App. B.3) */
  float *rho_prev;  /* [B,H,J,Dv]  TEMPORAL only: previous query prior rhobar_{t-1}       */
} swila_state_t;

/* Library version (major*10000 + minor*100 + patch). */
int swila_version(void);

/* Static, never-NULL description of a status code. */
const char *swila_strerror(int status);

/* Text of the most recent CUDA error seen by the calling thread ("" if none). */
const char *swila_last_cuda_error(void);

/* Device-side health of the current device: SWILA_OK, or SWILA_ERR_CUDA if a kernel of this
 * library gave up on a bounded wait since the last call (the flag is cleared).  Synchronises
 * the device; meant for tests and debugging, never needed on the normal path. */
int swila_device_status(void);

/* Bytes of state->W and of each of state->r_prev / state->rho_prev for `shape`
 * (0 if the shape is invalid). */
size_t swila_state_w_bytes(const swila_shape_t *shape);
size_t swila_state_r_bytes(const swila_shape_t *shape);

/* Initial state: W = 0 and, when TEMPORAL, r_prev = rho_prev = 1/J (the paper does not
 * state an initial distribution; uniform keeps both carried quantities distributions). */
int swila_state_init(const swila_shape_t *shape, swila_state_t *state, void *stream);

/*
 * Prefill: run the recurrence of Eqs. 3.3-3.5 (with the variants selected in
 * shape->flags) over all T tokens of q,k [B,H,T,Dk], v [B,H,T,Dv] and write o [B,H,T,Dv].
 *   state_in  : initial state; NULL means the state of swila_state_init.
 *   state_out : receives the state after token T; NULL discards it; may alias state_in
 *               (each thread block reads its slice completely before writing it).
 *   r_debug   : NULL, or fp32 [B,H,T,J,Dv] receiving the responsibilities r of Eq. 3.4.
 * T == 0 copies state_in to state_out and touches nothing else.
 * SWILA_ERR_ALIAS: o, r_debug or a tensor of state_out overlaps a streamed input (q, k, v, a gate tensor),
 * or o overlaps r_debug or the state; state_out may alias state_in only tensor for tensor, exactly.
 *
 * Which kernel runs (shape->algo).  Two kernels evaluate the same recurrence and agree to rounding
 * (1e-4 on the state):
 *   SCAN   the sequential scan on the FP32 ALUs: every shape, dtype, flag and output.
 *   CHUNK  32-token chunks whose state-times-token contractions run on the tcgen05 tensor cores (bf16
 *          hi/lo operand split, FP32 accumulation in tensor memory), the E-step and the corrections
 *          inside a chunk on the FP32 ALUs; several times faster.  It covers: bf16 io; Dk in {64, 128};
 *          not SWILA_QKV_ACT; and
 *            - ungated: J in {4, 8}, and J = 16 at Dk = 64; plain or SWILA_TEMPORAL; r_debug and the sums of
 *              swila_forward_stats for J <= 8;
 *            - SWILA_GATED with one decay per state row, SWILA_GATE_PER_OUT or SWILA_GATE_SCALAR, pre- or
 *              post-decay: J = 4, or J = 8 at Dk = 64; with SWILA_TEMPORAL at Dk = 64 only; no r_debug /
 *              statistics.  Such a
 *              call launches a guard pass over alpha, the chunked kernel and the scan kernel; exactly one of
 *              the two does the work: the scan if the product of some row's decays over a 32-token chunk is
 *              below 2^-40 (the chunked form divides by that product), which costs the scan's time.
 *          Requested for anything else (SWILA_GATE_PER_KEY and SWILA_GATE_ELEMENTWISE included: their decay
 *          differs per key dimension, so the rows of a tile share no operand): SWILA_ERR_UNSUPPORTED.
 *   AUTO   CHUNK when the call is inside that coverage and T >= 64, else SCAN.  So the following send an
 *          AUTO call to the scan kernel, at 3-6 times the cost per token: fp32 io, SWILA_QKV_ACT, Dk = 16,
 *          J in {1, 2}, T < 64, SWILA_GATED with per-key or elementwise decays or, at Dk = 128, with SWILA_TEMPORAL,
 *          and r_debug or statistics together with SWILA_GATED or J = 16.
 * Inside CHUNK the work distribution depends on state_out: with a state output, when the 128-row tiles
 * of the launch do not fill a whole number of waves of SMs, the chunk sequence is cut into equal runs
 * per SM and a tile that falls into two runs hands its state over through state_out (a cooperative
 * launch; hand-over flags live in a library array indexed by a launch counter modulo 8).  With
 * state_out == NULL every block takes whole tiles, which can cost up to one partly empty wave more.
 * Results are the same to rounding.
 *
 * The call only enqueues work on `stream`; it (and swila_decode_step) may be captured into a CUDA graph
 * and replayed, after one ordinary call of the same shape on the device.  Limits of a replayed CHUNK
 * launch with hand-over: a replay reuses the counter value of its capture, so it must not overlap on the
 * GPU another hand-over launch whose counter is congruent modulo 8 (in practice: do not overlap replays
 * with each other or with more than 7 live calls), and swila_device_status must be clean before a replay
 * (an expired wait leaves the launch incomplete).
 */
int swila_forward(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                  const swila_gates_t *gates, const swila_state_t *state_in,
                  swila_state_t *state_out, void *o, float *r_debug, void *stream);

/*
 * Sums over time of the mixture weights, for the mutual-information load-balancing loss (Sec. 3.5: entropy
 * of the time-averaged responsibilities minus the mean per-token entropy, key side and query side) and the
 * router diagnostics of App. D.5.  Every pointer is a DEVICE pointer to fp32 or NULL (that sum is not
 * formed).  The sums of a call are ADDED to the buffers, so a sequence fed in several calls accumulates;
 * the caller zeroes them first.
 */
typedef struct {
  float *r_sum;    /* [B,H,J,Dv] += sum over t of the responsibilities r_tjd of Eq. 3.4             */
  float *r_ent;    /* [B,H,Dv]   += sum over t of -sum_j r_tjd ln r_tjd (nats; 0 ln 0 = 0)          */
  float *rho_sum;  /* [B,H,J,Dv] += sum over t of the readout weights of Eq. 3.5: pi^q_tjd, or the  */
                   /*               running average rho-bar_tjd when TEMPORAL (App. B.3)            */
  float *rho_ent;  /* [B,H,Dv]   += sum over t of their entropy over j (nats)                       */
} swila_stats_t;

/*
 * swila_forward that also forms the sums of `stats` (which must not be NULL; any of its members may be).
 * The kernel is chosen as in swila_forward; outputs and state are those of swila_forward with the same
 * shape->algo, bit for bit.  The chunked kernel adds its sums with atomic operations (the pieces of a sequence
 * may run in different thread blocks), so their last bits can differ from run to run; the scan kernel's do not.
 */
int swila_forward_stats(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                        const swila_gates_t *gates, const swila_state_t *state_in,
                        swila_state_t *state_out, void *o, float *r_debug, const swila_stats_t *stats,
                        void *stream);

/*
 * RMSNorm of the layer output (App. D.1), in place: for every (batch, head, token) row of o [B,H,T,Dv]
 * (io dtype), o_d <- o_d / sqrt(mean over d of o_d^2 + eps) * weight_d.  weight: DEVICE fp32 [Dv], or NULL
 * for all ones.  A separate memory-bound pass over o (the rows of o are spread over several thread blocks
 * of the recurrence, so the mean is not available there).  Uses shape->B, H, T, Dv and io_dtype.
 */
int swila_output_norm(const swila_shape_t *shape, void *o, const float *weight, float eps, void *stream);

/*
 * Decode: one token of the same recurrence on a carried state, updated in place
 * (generation, App. D.4).  q,k [B,H,1,Dk]; v, o [B,H,1,Dv]; gate tensors with T = 1.
 * shape->T is ignored.  Decode always runs the scan kernel with T = 1 whatever shape->algo says
 * (SWILA_ALGO_CHUNK is read as SWILA_ALGO_SCAN): its arithmetic and order are those of a scan prefill,
 * so a scan prefill of T tokens equals, bit for bit, T decode steps; against a chunked prefill the two
 * agree to rounding (1e-4 on the state).
 */
int swila_decode_step(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                      const swila_gates_t *gates, swila_state_t *state, void *o, void *stream);

/*
 * Prefill with HOST buffers: the same computation as swila_forward (Eqs. 3.3-3.5), for callers
 * whose tensors live in host memory.  q, k, v, every pointer inside `gates`, `state_in`,
 * `state_out` and o are HOST pointers (pinned memory makes the copies asynchronous);
 * `workspace` is a DEVICE buffer of at least swila_forward_host_workspace_bytes(shape)
 * bytes, owned by the caller and reusable across calls.  The call enqueues the host-to-device
 * copies, the kernel(s), and the device-to-host copies of o and of the final state, and returns
 * without synchronising; everything is complete once `stream` has been synchronised.  Problems
 * of 64 MB and more go through in up to 8 slabs of (batch, head) pairs -- which are independent
 * -- with the copies on two internal streams (created on the first such call on a device and
 * kept) beside the kernels on `stream`, so that transfers in both directions overlap the
 * compute; `stream` waits for the internal streams at the end.  Smaller problems use `stream`
 * alone.  Calls from several host threads on one device are allowed (each with its own workspace):
 * they share those copy streams, and the library serialises their enqueue phases with a per-device lock.
 * state_in == NULL starts from the initial state; state_out == NULL discards the final state.
 * Errors as swila_forward, plus SWILA_ERR_SIZE when the workspace is too small.
 */
size_t swila_forward_host_workspace_bytes(const swila_shape_t *shape);
int swila_forward_host(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                       const swila_gates_t *gates, const swila_state_t *state_in,
                       swila_state_t *state_out, void *o, void *workspace, size_t workspace_bytes,
                       void *stream);

/*
 * swila_forward_host for callers that cannot allocate device memory (this entry point has no
 * counterpart in the paper; it computes exactly what swila_forward_host computes).
 *
 * Who needs it: code that is given host tensors and a stream but may not call cudaMalloc or
 * any allocating library routine -- a plug-in inside a host application with a fixed memory
 * budget, a callback running where allocation is forbidden.  Instead of a caller-supplied
 * workspace the call stages its inputs, state and output in a fixed array of
 * SWILA_STATIC_WORKSPACE_BYTES (16 MiB) that is part of the library image; every GPU that
 * loads the library holds that array until the process exits.  The call itself allocates
 * nothing and frees nothing.
 *
 *  - Size limit: the problem must satisfy swila_forward_host_workspace_bytes(shape) <=
 *    swila_forward_host_static_capacity(); larger problems are rejected with SWILA_ERR_SIZE
 *    before anything is enqueued.
 *  - First call on a device: looks up the array's device address (once per device, with that
 *    device current).  Make that first call outside any stream capture.
 *  - Sharing: all calls on a device use the same array and it keeps the previous call's bytes.
 *    That is harmless for sequential calls (each call overwrites what it reads), but two calls
 *    whose GPU work overlaps -- different streams, or different host threads -- race on it.
 *    Keep all calls to this entry point on one stream per device, or serialise them yourself.
 *  - All pointer arguments are HOST pointers as in swila_forward_host; results are complete
 *    once `stream` has been synchronised.
 */
#define SWILA_STATIC_WORKSPACE_BYTES (16u << 20)
size_t swila_forward_host_static_capacity(void);
int swila_forward_host_static(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                              const swila_gates_t *gates, const swila_state_t *state_in,
                              swila_state_t *state_out, void *o, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SWILA_H_ */
