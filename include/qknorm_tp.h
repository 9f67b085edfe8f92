/*
 * libqknorm, tensor-parallel entry points -- layerwise QK-RMSNorm when every rank
 * (GPU) holds one column slice of Q and of K, with the scalar exchange of Algorithm 1,
 * Phase B (Sections III-A to III-D of the paper).
 *
 * What a call computes on rank r (Algorithm 1, one kernel launch):
 *   Phase A   S_local[t]  = sum_j X_local[t][j]^2                (fp32)
 *   Phase B   push S_local[t] into every peer's inbox; wait until the N-1 peers'
 *             scalars for t have arrived in this rank's own inbox;
 *             S_global[t] = sum of the N scalars (fp32), added pairwise over the rank index
 *             (ranks 2i and 2i+1, then pairs of pairs, ...): the same tree on every rank,
 *             so every rank gets the same bits;
 *             RMS^-1      = 1 / sqrt(S_global / H_total + eps),  H_total = N * w
 *   Phase C   Y_local[t]  = (X_local[t] * W_local) * RMS^-1, rounded once, one write.
 * Per token, tensor and peer 8 bytes cross the link (Section III-A: scalars instead
 * of the O(H) activations an All-Gather would move).
 *
 * The inbox ("IPC buffer" of Algorithm 1).  Each rank owns one block of device
 * memory of qknorm_tp_inbox_bytes(N, token_capacity) bytes, on its own GPU, zeroed
 * ONCE before the first call and never cleared again.  Peers write into it, only its
 * owner reads it.  Layout: a 256-byte header (word 0: status, see qknorm_tp_status),
 * then 64-bit slots [parity 2][tensor 2][source rank N][token_capacity]; a slot holds
 * {epoch tag : 32, fp32 bits of the scalar : 32} and is written with one 64-bit store,
 * so value and "flag" cannot be seen apart.  A slot is "filled" for a call when its
 * tag equals the call's epoch.
 *
 * The epoch.  All ranks of a group make the same sequence of calls on the same
 * inboxes and number them alike: the first call has epoch 1, the next 2, and so on
 * (calls with tokens == 0 launch nothing and MUST NOT take a number).  Calls of one
 * rank on one inbox must be ordered (one stream, or events).  Consecutive epochs use
 * the two halves of the inbox in turn: a rank can be at most one call ahead of a
 * peer, so nothing needs clearing and no barrier is needed between calls.  Epoch 0 is
 * invalid (it is what a zeroed slot holds).  Before the 32-bit number wraps, all ranks
 * must quiesce, zero their inboxes and start again at 1.
 *
 * Launch.  Cooperative, so the driver refuses a grid whose CTAs cannot all be
 * resident: that is the bounded grid of Section III-D, under which a wait on a peer
 * cannot starve the CTA that would have served it.
 *
 * One GPU standing in for several.  `ranks` may describe n_local > 1 ranks whose
 * buffers all live on the current device; ONE launch then serves all of them (their
 * CTAs interleaved and co-resident), and peer_inbox[p] simply points at rank p's inbox
 * on the same device.  With n_local == num_ranks the call is self-contained; this is
 * how the protocol is tested on a single GPU.  With one process per GPU, n_local is 1
 * and peer_inbox[p] is a peer mapping of rank p's inbox (qknorm_tp_ipc_*).
 *
 * Every wait inside the kernel is bounded (wait_limit_us; 0 = one second).  If a
 * peer's scalar does not arrive in time the rank's kernel records the fact in its
 * inbox header and ends; the call has then produced undefined output for the tokens it
 * did not finish, the CUDA context stays usable, and qknorm_tp_status reports it.
 *
 * Conventions as in qknorm.h: data pointers are DEVICE pointers, pointer arrays and
 * descriptors are HOST memory read during the call only, the return value is a
 * qknorm_status, on error nothing was launched, tokens == 0 returns QKNORM_OK.
 * The vectorised path is the only one here: slice widths must be multiples of
 * 16 bytes, base pointers 16-byte aligned, pitches multiples of 16 bytes, and three
 * copies of a slice row pair (Q then K) plus the two gamma slices must fit a CTA's
 * shared memory (rows of up to about 60 KB); anything else is QKNORM_ERR_ALIGN /
 * QKNORM_ERR_SHAPE.
 */
#ifndef QKNORM_TP_H_
#define QKNORM_TP_H_

#include "qknorm.h"

#ifdef __cplusplus
extern "C" {
#endif

#define QKNORM_TP_IPC_HANDLE_BYTES 64

/* status word of an inbox (qknorm_tp_status) */
#define QKNORM_TP_STATUS_OK 0
#define QKNORM_TP_STATUS_PEER_TIMEOUT 1   /* a peer's scalar did not arrive within the limit */
#define QKNORM_TP_STATUS_STAGE_TIMEOUT 2  /* a bulk copy of the rank's own row did not complete within a second */

/* One rank's buffers.  X_local / W_local / Y_local of Algorithm 1 for Q and for K. */
typedef struct qknorm_tp_rank {
  int32_t rank;              /* 0 .. num_ranks-1 */
  int32_t reserved;          /* 0 */
  const void* q;             /* [tokens, wq] slice of Q, device, read  (ignored when wq == 0) */
  const void* k;             /* [tokens, wk] slice of K, device, read  (ignored when wk == 0) */
  const void* gamma_q;       /* [wq] bf16, device, read */
  const void* gamma_k;       /* [wk] bf16, device, read */
  void* out_q;               /* [tokens, wq], device, written; may equal q */
  void* out_k;               /* [tokens, wk], device, written; may equal k */
  float* rstd_q;             /* optional [tokens] fp32: RMS^-1 as this rank computed it */
  float* rstd_k;
  float* partial_q;          /* optional [tokens] fp32: this rank's own S_local */
  float* partial_k;
  void* inbox;               /* this rank's inbox, on this rank's GPU */
  const void* const* peer_inbox;  /* HOST array [num_ranks] of device pointers: rank p's inbox as the current
                                     device addresses it; entry [rank] is ignored */
} qknorm_tp_rank;

/* Bytes of one rank's inbox for num_ranks ranks and calls of up to token_capacity tokens. */
int qknorm_tp_inbox_bytes(int32_t num_ranks, int64_t token_capacity, int64_t* bytes);

/*
 * qknorm_fwd_tp / qknorm_fwd_tp_e4m3 -- Algorithm 1 for the n_local ranks described by
 * ranks[0 .. n_local-1] (bf16 activations, or FP8-E4M3 activations with bf16 gamma).
 *   wq, wk          slice widths in elements (H_total = num_ranks * w); one may be 0
 *   ld              NULL (contiguous rows) or HOST array {ld_q, ld_k, ld_out_q, ld_out_k} of row
 *                   pitches in elements, the same for every rank; an entry of 0 = contiguous
 *   token_capacity  what the inboxes were sized with; tokens <= token_capacity
 *   epoch           this call's number, see above; 0 is rejected
 *   wait_limit_us   bound of every wait on a peer, microseconds; 0 = 1,000,000
 * Errors: QKNORM_ERR_SHARDS for num_ranks or n_local outside 1..QKNORM_MAX_SHARDS, n_local >
 * num_ranks, a rank number outside 0..num_ranks-1 or listed twice; QKNORM_ERR_NULL,
 * _SHAPE, _ALIGN, _EPS as described above; QKNORM_ERR_ALIAS when an output overlaps
 * another buffer of the call (its own input excepted) or an inbox; QKNORM_ERR_CUDA when the
 * cooperative launch is refused.
 */
int qknorm_fwd_tp(const qknorm_tp_rank* ranks, int32_t n_local, int32_t num_ranks,
                  int64_t tokens, int64_t token_capacity, int32_t wq, int32_t wk, const int64_t* ld,
                  float eps, uint32_t epoch, uint32_t wait_limit_us, void* stream);
int qknorm_fwd_tp_e4m3(const qknorm_tp_rank* ranks, int32_t n_local, int32_t num_ranks,
                       int64_t tokens, int64_t token_capacity, int32_t wq, int32_t wk, const int64_t* ld,
                       float eps, uint32_t epoch, uint32_t wait_limit_us, void* stream);

/*
 * qknorm_tp_status -- copies the first four 32-bit words of an inbox header to out
 * (HOST pointer): {status, token at which the kernel gave up, rank whose scalar was
 * missing (-1 if not applicable), 0}.  Synchronous copy on the legacy default stream:
 * synchronise the stream of the call first.  qknorm_tp_clear_status zeroes the header
 * on `stream` so that the inbox can be used again once the group has recovered.
 */
int qknorm_tp_status(const void* inbox, int32_t* out);
int qknorm_tp_clear_status(void* inbox, void* stream);

/*
 * qknorm_tp_slot_index -- position (in 64-bit words from the start of an inbox) of the slot that
 * holds source rank `src_rank`'s scalar of token 0 for a call with this epoch; token t is t words
 * further.  tensor: 0 = Q, 1 = K.  Returns -1 for arguments out of range.
 * qknorm_tp_inbox_peek / _poke -- synchronous copies of n_words 64-bit words between an inbox (from
 * word first_word) and HOST memory: for tests, inspection and recovery tools (a slot is
 * (uint64_t)epoch << 32 | fp32 bits).  Not for use while a call on the inbox is in flight.
 */
int64_t qknorm_tp_slot_index(int32_t num_ranks, int64_t token_capacity, uint32_t epoch, int32_t tensor, int32_t src_rank);
int qknorm_tp_inbox_peek(const void* inbox, int64_t first_word, int64_t n_words, uint64_t* out);
int qknorm_tp_inbox_poke(void* inbox, int64_t first_word, int64_t n_words, const uint64_t* in);

/*
 * Inbox management for one process per GPU.  These are the only routines of the
 * library that allocate or map device memory, and none of them is called by the
 * forward entry points.
 *   qknorm_tp_inbox_create   cudaMalloc on the current device + zero fill (synchronous).
 *   qknorm_tp_inbox_zero     zero fill of the whole inbox on `stream` (asynchronous): for the restart
 *                            before the epoch wraps, after all ranks have quiesced.
 *   qknorm_tp_inbox_destroy  cudaFree.
 *   qknorm_tp_ipc_export     inter-process handle (64 bytes, HOST buffer) of an inbox made by
 *                            qknorm_tp_inbox_create; send it to the peers by any host channel.
 *   qknorm_tp_ipc_open       maps a peer's inbox into this process on the current device
 *                            (peer access over NVLink); *out is the pointer for peer_inbox[p].
 *   qknorm_tp_ipc_close      unmaps it.
 */
int qknorm_tp_inbox_create(int32_t num_ranks, int64_t token_capacity, void** out);
int qknorm_tp_inbox_zero(void* inbox, int32_t num_ranks, int64_t token_capacity, void* stream);
int qknorm_tp_inbox_destroy(void* inbox);
int qknorm_tp_ipc_export(const void* inbox, unsigned char* handle);
int qknorm_tp_ipc_open(const unsigned char* handle, void** out);
int qknorm_tp_ipc_close(void* mapped);

#ifdef __cplusplus
}
#endif
#endif /* QKNORM_TP_H_ */
