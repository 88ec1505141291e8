/*
 * swila_dev.h -- developer entry points of libswila.so: a measurement helper, self-tests of the
 * tensor-core plumbing and host-only probes of the chunked kernel's work distribution.  None of
 * them is part of the recurrence and none has a counterpart in the paper; the product's C ABI is
 * swila.h.  They are exported so that the benchmark harness and the tests can reach them through
 * the same library.
 *
 * Conventions as in swila.h: DEVICE pointers unless a function says HOST, asynchronous on
 * `stream`, SWILA_OK or a negative swila_status code.
 */
#ifndef SWILA_DEV_H_
#define SWILA_DEV_H_

#include "swila.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Measurement helper (no counterpart in the paper): launches an FP32 FMA-chain
 * microbenchmark whose rate is the denominator of the scan kernel's roofline (the
 * recurrence costs 3*J*Dk*Dv FP32 FMAs per token and head, Sec. 3.2).  Every thread of
 * `blocks` blocks of 256 threads runs `iters` rounds of 2*`chains` independent register
 * FMAs; packed != 0 uses the packed f32x2 form.  chains in {4, 8, 16}.  scratch_out: device
 * pointer to >= 4 bytes (practically never written).  *fma_per_launch (HOST pointer) receives
 * the number of FMAs one launch performs; time the launch with CUDA events on `stream`.
 */
int swila_bench_fma_chain(int packed, int chains, int blocks, int iters, float *scratch_out,
                          double *fma_per_launch, void *stream);

/*
 * Self-test of the tensor-core plumbing (no counterpart in the paper): one block computes
 * D[128 x N] = A[128 x K] * B[N x K]^T with TF32 operands and FP32 accumulation on the tcgen05
 * path (A through tensor memory, B through shared memory).  A [128,K], B [N,K], D [128,N] are
 * DEVICE fp32 row-major; *status (DEVICE int, zeroed by the caller) is set non-zero if the MMA
 * never completed.  (N, K) in {(32,32), (128,32), (32,128), (64,128)}.
 */
int swila_selftest_tf32_mma(const float *A, const float *B, float *D, int N, int K, int *status, void *stream);

/*
 * The same self-test with BF16 operands (no counterpart in the paper): A and B are DEVICE fp32
 * row-major and are rounded to bf16 (nearest even) by the kernel; FP32 accumulation.  a_in_smem = 0:
 * A goes through tensor memory, two consecutive K elements per 32-bit column; a_in_smem = 1: A
 * goes through shared memory in the K-major layout of B; a_in_smem = 2: both operands in shared
 * memory in the 128-byte-swizzle K-major layout (what a tensor copy with that swizzle mode
 * writes); a_in_smem = 3: A through tensor memory, B stored MN-major (N contiguous) with the
 * 128-byte swizzle.  (N, K, a_in_smem) in {(64,128,0), (128,32,0), (32,32,0), (64,64,1),
 * (64,64,2), (32,64,2), (128,32,3)}; anything else returns SWILA_ERR_UNSUPPORTED.
 */
int swila_selftest_bf16_mma(const float *A, const float *B, float *D, int N, int K, int a_in_smem, int *status,
                            void *stream);

/*
 * Self-test of the failure path of the chunked kernel's waits (no counterpart in the paper): launches one small block
 * that waits, with the library's bounded wait (about two seconds), on a barrier nothing arrives at.  The wait must
 * give up and the kernel end normally; *gave_up (DEVICE int) receives 1, and the next swila_device_status() reports
 * SWILA_ERR_CUDA once (then SWILA_OK again).  Nothing traps or faults: the context stays usable.
 */
int swila_selftest_wait_timeout(int *gave_up, void *stream);

/*
 * Which kernel SWILA_ALGO_AUTO resolves to for `shape` (no counterpart in the paper; host arithmetic only):
 * returns SWILA_ALGO_CHUNK or SWILA_ALGO_SCAN, or a negative status for an invalid shape.  aux_outputs != 0: the
 * call also asks for r_debug or for the sums of swila_forward_stats.  The rule is the one stated with swila_forward.
 */
int swila_auto_algo(const swila_shape_t *shape, int aux_outputs);

/*
 * Host-only probes of how SWILA_ALGO_CHUNK distributes work (no counterpart in the paper; no GPU call).
 * A launch has B*H*ceil(Dv / (128/J)) tiles of 128 state rows, each a sequence of ceil(T/32) chunks.
 *
 * swila_chunk_plan: the layout chosen for a device with `sm_count` SMs.  out[0] = 1 if the chunk sequence
 * is cut into equal runs (taken when the tiles do not fill a whole number of waves and a state output is
 * given), else 0 (one tile per block); out[1] = blocks per gang (column slices of one (batch, head));
 * out[2] = chunks per unit; out[3] = chunks per run; out[4] = units (tiles, or (batch, head) pairs when
 * split); out[5] = blocks launched.  Returns SWILA_OK or an error code (J must be 4 or 8).
 *
 * swila_chunk_run_pieces: the pieces of run `run` in the order a block processes them, as triples
 * (unit, first chunk, end chunk) written to `pieces` (HOST int[3 * capacity]).  Returns the number of pieces
 * (0 for a run past the end of the work) or a negative error code.
 */
int swila_chunk_plan(int B, int H, int T, int Dv, int J, int sm_count, int has_state_out, long long out[6]);
int swila_chunk_run_pieces(long long units, int nch, int per, long long run, int *pieces, int capacity);

#ifdef __cplusplus
}
#endif
#endif /* SWILA_DEV_H_ */
