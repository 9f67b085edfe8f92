/*
 * libqknorm -- layerwise Query-Key RMSNorm for NVIDIA B200 (sm_100a).
 *
 * The operation (Eq. 1 of the paper, Section II-A): every token's full
 * projected Q vector, and separately its full K vector, is replaced by
 *
 *     y[j] = x[j] / sqrt( (1/H) * sum_j x[j]^2 + eps ) * gamma[j]
 *
 * with H the FULL width of that vector (dq for Q, dk for K), one statistic per
 * token per tensor ("layerwise": one factor for the whole vector, not one per
 * head).  The statistic is formed the way Algorithm 1 forms it: a per-shard
 * partial sum of squares in fp32 (Phase A), the partials combined as scalars in
 * ascending shard order in fp32 (Phase B, "P2P reduction"),
 * rstd = 1/sqrt(S_global/H_total + eps), and a single write of
 * (x * gamma) * rstd (Phases B/C).  On one GPU the shards are logical: separate
 * device buffers that hold equal contiguous column slices.
 *
 * Conventions for every entry point
 *  - Data pointers are DEVICE pointers.  Activations and gammas are bf16 stored
 *    as 16-bit words; rows are contiguous (leading dimension = width).
 *  - Pointer ARRAYS (the *_shards arguments) are HOST arrays of device pointers.
 *    They are read during the call only and may be freed on return.
 *  - Ownership: the caller owns every buffer.  The library allocates nothing on
 *    the device and frees nothing.  Its own state: a per-device cache of the SM
 *    count and kernel occupancy on the host, and a few KB of device memory inside
 *    the library image (an error word; 256 token counters, one per stream that has
 *    made a prefill-size call, each back at zero when its kernel ends).
 *  - Asynchrony: work is enqueued on `stream` (a cudaStream_t passed as void*;
 *    NULL = the legacy default stream) and the call returns without
 *    synchronising.  No cudaMalloc, no cudaMemcpy, no host synchronisation.
 *    Decode-size and prefill-size calls are launched with programmatic stream
 *    serialisation: the launch may begin while the previous kernel of the stream is still
 *    running, and the kernel waits for that kernel to complete (and its writes to be
 *    visible) before its first memory access, so stream order is kept as usual.
 *    Calls on different streams may run at the same time; calls may be captured into
 *    CUDA graphs.
 *  - Errors: the return value is a qknorm_status.  On any error nothing has
 *    been launched.  tokens == 0 returns QKNORM_OK without a launch.
 *  - A tensor can be skipped: dq == 0 (with its pointers ignored) means "K
 *    only", dk == 0 means "Q only".
 *  - Aliasing: an output may be exactly its own input (in-place, per shard).
 *    Any other overlap between an output and any other buffer of the call is
 *    rejected with QKNORM_ERR_ALIAS.
 *  - Precision: inputs are widened to fp32 (exact), sums of squares and all
 *    arithmetic are fp32, the product x*gamma*rstd is rounded ONCE to bf16
 *    (round to nearest even).  Subnormals are kept.  Results are bitwise
 *    reproducible run to run: prefill-size calls hand tokens to warps through a
 *    counter, but a token's arithmetic does not depend on the warp that does it,
 *    and no value is ever accumulated with atomics.
 *  - Fast path: when every base pointer is 16-byte aligned and every (shard)
 *    width is a multiple of 8 elements, vectorised kernels run; any other
 *    width or alignment is served by a slower general kernel, not an error.  A call is
 *    one kernel launch, except for some very wide rows (Q and K together beyond 32768
 *    elements, or beyond 10240 elements in 8 or more slices with K much narrower than Q):
 *    there Q and K, whose statistics are independent, get a launch each.
 */
#ifndef QKNORM_H_
#define QKNORM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QKNORM_MAX_DIM 65536   /* largest dq or dk */
#define QKNORM_MAX_SHARDS 16   /* largest num_shards */

typedef enum {
  QKNORM_OK = 0,
  QKNORM_ERR_NULL = 1,    /* a required pointer is NULL */
  QKNORM_ERR_SHAPE = 2,   /* tokens < 0, a width < 0 or > QKNORM_MAX_DIM, width not divisible by num_shards, or dq == dk == 0 with tokens > 0 */
  QKNORM_ERR_ALIGN = 3,   /* a bf16 pointer is not 2-byte aligned, or an fp32 pointer not 4-byte aligned */
  QKNORM_ERR_ALIAS = 4,   /* an output overlaps another buffer without being exactly its own input */
  QKNORM_ERR_SHARDS = 5,  /* num_shards < 1 or > QKNORM_MAX_SHARDS */
  QKNORM_ERR_EPS = 6,     /* eps < 0 or NaN */
  QKNORM_ERR_CUDA = 7,    /* a CUDA call failed; see qknorm_last_cuda_error() */
  QKNORM_ERR_HEADS = 8,   /* head_dim < 1 or does not divide dq (or dk) */
  QKNORM_ERR_SCRATCH = 9,       /* scratch buffer NULL, too small, misaligned, or overlapping a buffer of the call */
  QKNORM_ERR_STATIC_LIMIT = 10  /* the call needs more scratch than the library's built-in array holds */
} qknorm_status;

/*
 * qknorm_fwd -- Eq. 1 on unsharded rows (the problem statement of Section II-A;
 * Algorithm 1 with N = 1).
 *   q        [tokens, dq] bf16, device, read      k        [tokens, dk] bf16, device, read
 *   gamma_q  [dq] bf16, device, read              gamma_k  [dk] bf16, device, read
 *   out_q    [tokens, dq] bf16, device, written   out_k    [tokens, dk] bf16, device, written
 *   out_q may equal q and out_k may equal k (in place).
 */
int qknorm_fwd(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
               int64_t tokens, int32_t dq, int32_t dk, float eps,
               void* out_q, void* out_k, void* stream);

/*
 * qknorm_fwd_sharded -- the same result when each row is held as num_shards
 * equal column slices in separate buffers (Section III-A, Algorithm 1 Phases
 * A-C with N = num_shards logical ranks on one GPU).  Slice s holds columns
 * [s*w, (s+1)*w) of the full row, w = dq/num_shards (resp. dk/num_shards);
 * gamma is sliced the same way (W_local of Algorithm 1).  dq and dk are the FULL
 * widths (H_total): the mean is over the whole vector.
 *   q_shards, k_shards, gamma_q_shards, gamma_k_shards, out_q_shards, out_k_shards:
 *     HOST arrays of num_shards device pointers; q_shards[s] is [tokens, dq/num_shards], etc.
 *   out_*_shards[s] may equal the matching input shard (in place).
 */
int qknorm_fwd_sharded(const void* const* q_shards, const void* const* k_shards,
                       const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                       int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                       void* const* out_q_shards, void* const* out_k_shards, void* stream);

/*
 * The *_ex forms run the same kernels and additionally store the statistic, so
 * that tests can check it on its own (Algorithm 1: S_local, RMS^-1).
 *   rstd_q, rstd_k         [tokens] fp32, device, written; NULL = not wanted
 *   partials_q, partials_k [num_shards, tokens] fp32, device, written; NULL = not wanted.
 *                          partials[s*tokens + t] is shard s's own sum of squares for token t
 *                          (the scalar each rank would publish in Phase A).
 */
int qknorm_fwd_ex(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                  int64_t tokens, int32_t dq, int32_t dk, float eps,
                  void* out_q, void* out_k, float* rstd_q, float* rstd_k, void* stream);

int qknorm_fwd_sharded_ex(const void* const* q_shards, const void* const* k_shards,
                          const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                          int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                          void* const* out_q_shards, void* const* out_k_shards,
                          float* partials_q, float* partials_k, float* rstd_q, float* rstd_k,
                          void* stream);

/*
 * qknorm_fwd_strided -- qknorm_fwd on rows that are not contiguous: row t of q starts
 * ld_q ELEMENTS after row t-1 (ld_q >= dq), likewise k, out_q, out_k; 0 means
 * contiguous (ld = width).  This is the layout between the projection and attention
 * (Section II-A) when Q and K are column blocks of one fused [tokens, dq + 2*dk]
 * projection output: q = base, k = base + dq, ld_q = ld_k = dq + 2*dk.  In place
 * (out == in with the same ld) is allowed; the Q and K views of one buffer do not
 * count as overlapping.  bf16; the vectorised kernels also need every ld to be a
 * multiple of 8 elements.  A negative ld or ld < width is QKNORM_ERR_SHAPE.
 */
int qknorm_fwd_strided(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                       int64_t tokens, int32_t dq, int32_t dk, int64_t ld_q, int64_t ld_k, float eps,
                       void* out_q, void* out_k, int64_t ld_out_q, int64_t ld_out_k, void* stream);

/* qknorm_fwd_strided with FP8-E4M3 activations (one byte per element, gamma bf16; see
 * qknorm_fwd_e4m3).  Strides are in elements; the vectorised kernels need every ld to be a
 * multiple of 16 elements. */
int qknorm_fwd_strided_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                            int64_t tokens, int32_t dq, int32_t dk, int64_t ld_q, int64_t ld_k, float eps,
                            void* out_q, void* out_k, int64_t ld_out_q, int64_t ld_out_k, void* stream);

/*
 * qknorm_fwd_headwise -- the other granularity Section II-A names, headwise: every
 * attention head gets a normalisation factor of its own.  Row t of q is cut into
 * dq/head_dim heads of head_dim consecutive columns; every head is normalised on its
 * own, y = x / sqrt(mean over the head of x^2 + eps) * gamma, with the gamma entries of
 * its columns (gamma_q has dq entries; tile a [head_dim] weight if the model shares
 * it between heads).  Likewise k.  A head never straddles a tensor-parallel shard, so
 * nothing is combined across shards.
 *   ld_*            row strides in elements as in qknorm_fwd_strided (0 = contiguous)
 *   rstd_q, rstd_k  optional [tokens, dq/head_dim] / [tokens, dk/head_dim] fp32, device
 * head_dim < 1 or not dividing a (shard) width is QKNORM_ERR_HEADS.  Vectorised for heads
 * of a multiple of 16 bytes up to 512 bytes with 16-byte aligned pointers and strides; any
 * other head_dim or alignment takes a general kernel.
 *   qknorm_fwd_headwise                bf16 rows, optional strides
 *   qknorm_fwd_headwise_e4m3           the same with q, k and the outputs as FP8-E4M3 (gamma bf16)
 *   qknorm_fwd_headwise_sharded        the tensors as num_shards column slices (host arrays of
 *                                      device pointers as in qknorm_fwd_sharded, contiguous rows):
 *                                      all slices in ONE launch; dq, dk are the FULL widths;
 *                                      rstd column s * (heads per slice) + h is head h of slice s
 *   qknorm_fwd_headwise_sharded_e4m3   the same for FP8-E4M3
 */
int qknorm_fwd_headwise(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                        int64_t tokens, int32_t dq, int32_t dk, int32_t head_dim,
                        int64_t ld_q, int64_t ld_k, float eps, void* out_q, void* out_k,
                        int64_t ld_out_q, int64_t ld_out_k, float* rstd_q, float* rstd_k, void* stream);
int qknorm_fwd_headwise_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                             int64_t tokens, int32_t dq, int32_t dk, int32_t head_dim,
                             int64_t ld_q, int64_t ld_k, float eps, void* out_q, void* out_k,
                             int64_t ld_out_q, int64_t ld_out_k, float* rstd_q, float* rstd_k, void* stream);
int qknorm_fwd_headwise_sharded(const void* const* q_shards, const void* const* k_shards,
                                const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, int32_t head_dim,
                                float eps, void* const* out_q_shards, void* const* out_k_shards,
                                float* rstd_q, float* rstd_k, void* stream);
int qknorm_fwd_headwise_sharded_e4m3(const void* const* q_shards, const void* const* k_shards,
                                     const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                     int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk,
                                     int32_t head_dim, float eps, void* const* out_q_shards,
                                     void* const* out_k_shards, float* rstd_q, float* rstd_k, void* stream);

/*
 * FP8-E4M3 activations (Section IV-C: the local sums of squares and the reduction of the
 * scalars across shards stay in fp32 whatever format the activations are stored in).
 * The same operation with q, k and the outputs stored as FP8 E4M3 (one byte per
 * element: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities,
 * S.1111.111 = NaN, largest finite value 448).  gamma stays bf16; all arithmetic is
 * fp32; the result is rounded once to E4M3, to nearest even, saturating at +-448.
 * Arguments as qknorm_fwd_ex / qknorm_fwd_sharded_ex (rstd_* and partials_* may be
 * NULL).  Vectorised kernels need 16-byte aligned pointers and (shard) widths that
 * are multiples of 16 elements; other shapes take the general kernel.
 */
int qknorm_fwd_e4m3(const void* q, const void* k, const void* gamma_q, const void* gamma_k,
                    int64_t tokens, int32_t dq, int32_t dk, float eps,
                    void* out_q, void* out_k, float* rstd_q, float* rstd_k, void* stream);

int qknorm_fwd_sharded_e4m3(const void* const* q_shards, const void* const* k_shards,
                            const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                            int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                            void* const* out_q_shards, void* const* out_k_shards,
                            float* partials_q, float* partials_k, float* rstd_q, float* rstd_k,
                            void* stream);

/*
 * One-GPU stand-ins for the two conventional ways of doing tensor-parallel QK-Norm
 * that the paper measures against (Section II-C, Section IV-A "Baselines"), for
 * quoting the fused path in the paper's terms.  Same arguments and the same result
 * as qknorm_fwd_sharded (bf16, contiguous rows, in place allowed), plus a scratch
 * buffer in DEVICE memory that the caller owns; it must not overlap any buffer of
 * the call (QKNORM_ERR_SCRATCH otherwise, also when it is NULL, misaligned or too
 * small).  Its contents after the call are unspecified.
 *
 * qknorm_baseline_gather_then_norm -- "All-Gather, then RMSNorm": one kernel copies
 *   the num_shards slices of every row side by side into scratch (full rows, what
 *   every rank would hold after the All-Gather), then the normalisation runs with
 *   the scratch as its input.  Two launches; every activation crosses HBM four
 *   times.  scratch: tokens * (dq + dk) * 2 bytes, 16-byte aligned.
 * qknorm_baseline_two_pass -- scalar aggregation without fusion: a statistics
 *   kernel writes every slice's sum of squares to scratch (the scalars a rank would
 *   send), a second kernel adds them in ascending slice order and scales.  Two
 *   launches; every activation is read twice and written once.
 *   scratch: 2 * num_shards * tokens floats.
 */
int qknorm_baseline_gather_then_norm(const void* const* q_shards, const void* const* k_shards,
                                     const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                     int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                                     void* const* out_q_shards, void* const* out_k_shards,
                                     void* scratch, size_t scratch_bytes, void* stream);

int qknorm_baseline_two_pass(const void* const* q_shards, const void* const* k_shards,
                             const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                             int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                             void* const* out_q_shards, void* const* out_k_shards,
                             float* scratch, size_t scratch_bytes, void* stream);

/*
 * qknorm_baseline_two_pass_static -- qknorm_baseline_two_pass for callers that cannot
 * bring a scratch buffer.  (The paper has no counterpart; this is a convenience of
 * this library.)
 *
 * Who needs it: code that must not allocate device memory where it makes the call.
 * Typical cases are a serving engine that has already handed all free HBM to its
 * KV-cache pool, so that a cudaMalloc for a few hundred kilobytes would fail or force
 * the pool to shrink, and a plug-in that runs inside someone else's step loop, where
 * cudaMalloc/cudaFree would stall the whole device and the host framework's allocator
 * is not reachable from C.  This entry point calls no cudaMalloc, no cudaFree and no
 * library routine that allocates.
 *
 * How: the statistics pass writes every slice's sum of squares into an array that is
 * part of the library image itself (static device memory, 262144 floats = 1 MiB; every
 * GPU that loads the library holds that 1 MiB until the process exits), and the scale
 * pass reads them back.  Arguments and result are those of qknorm_baseline_two_pass
 * without the scratch arguments.
 *
 * Limits and rules:
 *  - 2 * num_shards * tokens must not exceed qknorm_static_scratch_capacity()
 *    (262144), else QKNORM_ERR_STATIC_LIMIT and nothing is launched.  Split the tokens
 *    over several calls, or use qknorm_baseline_two_pass with your own buffer.
 *  - The first call on each device looks up the array's device address
 *    (cudaGetSymbolAddress, with that device current) and keeps it; make that first call
 *    before any stream capture begins on that device.
 *  - All calls on a device share the one array, and it keeps whatever the last call
 *    left in it.  Nothing needs clearing between calls (a call only reads back what its
 *    own first pass wrote), but two calls that can overlap on the GPU -- different
 *    streams, or the same stream with programmatic overlap -- race on it and give wrong
 *    results.  Serialise them.
 */
int qknorm_baseline_two_pass_static(const void* const* q_shards, const void* const* k_shards,
                                    const void* const* gamma_q_shards, const void* const* gamma_k_shards,
                                    int32_t num_shards, int64_t tokens, int32_t dq, int32_t dk, float eps,
                                    void* const* out_q_shards, void* const* out_k_shards, void* stream);

/* Number of floats in the built-in scratch array of qknorm_baseline_two_pass_static. */
int64_t qknorm_static_scratch_capacity(void);

/* Human-readable name of a qknorm_status (static storage, never NULL). */
const char* qknorm_status_string(int status);

/* The cudaError_t of the last failing CUDA call made by this thread inside the
 * library (0 if none). */
int qknorm_last_cuda_error(void);

/* Debugging aid; SYNCHRONISES the device.  Every wait inside a kernel of this
 * library is bounded; a wait that ran out makes its CTA leave early and sets a
 * per-device error word.  This call copies that word to *out (host pointer):
 * 0 = no wait ever ran out on the current device since the library was loaded. */
int qknorm_device_error_word(int* out);

/* Name of the kernel variant the last successful call on this thread launched
 * ("warp", "tile", "ring", "rows", "wide", "general", "head", "head_general", "two_pass", "tp", "none"); static storage.  For tests and benchmarks. */
const char* qknorm_last_variant(void);

/* Number of kernel launches this thread has enqueued through the library. */
int64_t qknorm_launch_count(void);

/* Library version: major*10000 + minor*100 + patch. */
int qknorm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QKNORM_H_ */
