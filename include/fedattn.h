/*
 * fedattn.h -- C ABI of the FedAttn attention hot path for NVIDIA B200 (sm_100a).
 *
 * FedAttn (federated attention): N participants each hold a contiguous segment of a global
 * token sequence.  In most Transformer blocks every participant runs causal self-attention
 * over its own segment only (fedattn_local).  Every H-th block the participants' K/V are
 * aggregated -- concatenated in participant order, or sparsified (fedattn_aggregate_kv) --
 * and each participant's queries attend over the aggregated KV under the global-position
 * causal mask (fedattn_sync).  Cached K/V are reused for one-token decoding (fedattn_decode).
 *
 * Conventions for every call
 *   - "dev" pointers are device memory on the context's device; "host" pointers are ordinary
 *     host memory that is read before the call returns.  The caller owns every buffer,
 *     including the workspace.  Unless a function says otherwise it allocates nothing and
 *     frees nothing.
 *   - Work is enqueued on the given stream (a cudaStream_t passed as void*; NULL = default
 *     stream) and the call returns without synchronising.
 *   - Errors are return codes.  Arguments are validated on the host before anything is
 *     launched; a rejected call launches nothing.  A device-side anomaly (a bounded wait that
 *     ran out, an out-of-range or unsorted index in INDEXED mode, positions in an order the call
 *     cannot handle) sets a status word in the workspace that fedattn_poll reads; the kernel still
 *     terminates and the context stays usable.  Outputs of the call that raised the status are
 *     undefined.  After FEDATTN_ERR_TIMEOUT the bf16 head_dim 128 attention calls enqueued before
 *     the next fedattn_poll do no work and leave their outputs untouched (they would otherwise
 *     each wait out the same limit); poll, then repeat them.
 *   - Q, K and V must be finite.  Rows outside a query's allowed set carry weight exactly 0, but
 *     a tile that straddles a segment boundary multiplies those weights with the neighbour's V
 *     rows, and 0 * Inf or 0 * NaN is NaN.
 *   - Layouts are row-major with head_dim contiguous.  Packed queries Q[L, Hq, d]; packed keys
 *     and values K,V[L, Hkv, d]; L = sum of segment lengths; query head h reads KV head
 *     h / (Hq / Hkv).  dtype is FEDATTN_F32 or FEDATTN_BF16 for all of Q, K, V, O of a call;
 *     lse is always float.  Softmax and accumulation are fp32.
 *   - One context serves one stream at a time: calls that share a context and may overlap on
 *     the GPU race on its workspace.
 *   - Results are those of stream order: every call behaves as if it ran after all earlier work
 *     of its stream and before all later work.  fedattn_decode and the sparse modes of
 *     fedattn_aggregate_kv are launched with programmatic stream serialization and may touch
 *     their buffers before the preceding kernel of the stream has ended; the library tracks the
 *     buffers of such calls and holds a call back whenever that could be observed.  What the
 *     caller has to keep: a kernel of the caller's own that is launched with the programmatic
 *     attribute into the same stream executes griddepcontrol.wait before it ends (kernels
 *     launched the ordinary way need nothing), and buffers shared with work on OTHER streams are
 *     ordered by events or stream synchronisation, as always.
 */
#ifndef FEDATTN_H_
#define FEDATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FEDATTN_MAX_PARTICIPANTS 64
#define FEDATTN_MAX_HEAD_DIM 128

typedef struct fedattn_ctx fedattn_ctx; /* opaque */
typedef void *fedattn_stream;           /* a cudaStream_t */

typedef enum {
    FEDATTN_OK = 0,
    FEDATTN_ERR_INVALID_ARG = 1, /* null pointer, bad shape, non-monotone cu_seqlens, k_sel > L_n ... */
    FEDATTN_ERR_UNSUPPORTED = 2, /* valid request this build has no kernel for */
    FEDATTN_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
    FEDATTN_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed */
    FEDATTN_ERR_TIMEOUT = 5,     /* device status: a bounded wait inside a kernel ran out */
    FEDATTN_ERR_INDEX = 6,       /* device status: INDEXED selection index out of range or not ascending */
    FEDATTN_ERR_ORDER = 7        /* device status: kv_pos not non-decreasing in a call that needs it */
} fedattn_status;

typedef enum { FEDATTN_F32 = 0, FEDATTN_BF16 = 1 } fedattn_dtype;

typedef struct {
    int32_t n_participants; /* N, 1..FEDATTN_MAX_PARTICIPANTS */
    int32_t n_q_heads;      /* Hq */
    int32_t n_kv_heads;     /* Hkv, divides Hq */
    int32_t head_dim;       /* d, multiple of 8, <= FEDATTN_MAX_HEAD_DIM */
    int32_t dtype;          /* fedattn_dtype */
    int32_t causal;         /* 1 = decoder (masked) attention, 0 = bidirectional */
    float scale;            /* softmax scale; 0 selects 1/sqrt(head_dim) */
} fedattn_shape;

/* ---- context ------------------------------------------------------------------------------ */

/* Bytes of workspace the calls below need for this shape when no call handles more than
 * max_total_tokens query rows or max_total_kv aggregated KV rows.  Returns 0 for a bad shape. */
size_t fedattn_workspace_bytes(const fedattn_shape *shape, int64_t max_total_tokens,
                               int64_t max_total_kv);

/* Creates a context on `device` around a caller-owned dev workspace (256-byte aligned).  The
 * workspace's first bytes hold the device status word, which this call clears (the only
 * synchronous device operation besides fedattn_poll).  Host memory for the context itself is
 * allocated here and released by fedattn_destroy; the workspace is never freed. */
fedattn_status fedattn_create(fedattn_ctx **ctx, int device, void *workspace, size_t workspace_bytes);
void fedattn_destroy(fedattn_ctx *ctx);
const char *fedattn_status_string(fedattn_status s);

/* Synchronises `stream`, returns the device status word (FEDATTN_OK when no kernel reported
 * an anomaly) and clears it. */
fedattn_status fedattn_poll(fedattn_ctx *ctx, fedattn_stream stream);

/* Number of kernels this context has launched so far (for launch accounting), and how many of
 * them were launches of the tensor-core (tcgen05) attention kernel. */
int64_t fedattn_launch_count(const fedattn_ctx *ctx);
int64_t fedattn_tensor_core_launch_count(const fedattn_ctx *ctx);

/* Self-test of the bounded-wait protocol that every in-kernel wait follows.  Launches one small
 * kernel that waits, with the library's own wait routine and a limit of `max_polls` polls
 * (1..65536), on a barrier that nothing ever signals.  The wait runs out, the kernel raises
 * FEDATTN_ERR_TIMEOUT in the status word and returns normally: no trap, no fault, the context
 * stays usable.  For tests of the poll-and-repeat protocol described above. */
fedattn_status fedattn_selftest_wait_timeout(fedattn_ctx *ctx, int32_t max_polls, fedattn_stream stream);

/* ---- local attention: Phase I, o_n = Attention(q_n, k_n, v_n) ----------------------------------
 * Paper: Sec. IV-B "Phase I: Local Self-Attention", eq. (update_local_o), Algorithm 1 inner loop;
 * causal mask of Sec. III-B read as "key j allowed for query i iff j <= i" (self included).
 * Row i of segment n (cu_seqlens[n] <= i < cu_seqlens[n+1]) attends keys cu_seqlens[n] .. i
 * (the whole segment when shape->causal == 0).
 *   q dev [L,Hq,d]; k, v dev [L,Hkv,d]; cu_seqlens_host host int32 [N+1], cu[0] = 0, non-decreasing,
 *   cu[N] = L (zero-length segments allowed); o dev [L,Hq,d] written; lse dev float [L,Hq] or NULL
 *   (natural-log-sum-exp of the scaled logits). */
fedattn_status fedattn_local(fedattn_ctx *ctx, const fedattn_shape *shape,
                             const void *q, const void *k, const void *v,
                             const int32_t *cu_seqlens_host,
                             void *o, float *lse, fedattn_stream stream);

/* ---- KV aggregation: [K V] = sum_n Pi_n [k_n v_n] ---------------------------------------------
 * Paper: Sec. IV-B Phase II eq. (update_global_kv_H), Algorithm 1 exchange step (dense); Sec. V
 * Observation "Aggregation method": sparse KV exchange / adaptive KV aggregation pi_n(t) with
 * L'_n(t) subset of L_n (TOPK_KNORM, INDEXED; k_sel[n] = 0 excludes participant n).
 *
 *   FEDATTN_AGG_CONCAT      k_agg, v_agg dev [L,Hkv,d]: participant n's rows copied to rows
 *                           off_n .. off_n+L_n-1.  kv_pos dev int32 [L] = 0..L-1.  cu_kv = off.
 *   FEDATTN_AGG_TOPK_KNORM  per participant and per KV head keep the k_sel[n] rows with the
 *                           largest score s = sum_c k[j,h,c]^2 (fp64, c increasing); equal scores:
 *                           lower index first.  Kept rows are emitted in ascending index order.
 *   FEDATTN_AGG_INDEXED     as TOPK but the kept local indices are given in sel_idx_in
 *                           (dev int32 [Hkv, T], T = sum k_sel, block n at cu_kv[n], ascending).
 *   FEDATTN_AGG_TOPK_TOKEN  token-level selection (the selection matrix pi_n picks whole tokens):
 *                           one score per token, the squared norm of its whole key row [Hkv*d]
 *                           (fp64, memory order), same tie rule; every KV head keeps the same
 *                           tokens.  Outputs are token-major: k_agg, v_agg dev [T, Hkv, d];
 *                           kv_pos dev int32 [T]; sel_idx_out dev int32 [T]; to be passed to
 *                           fedattn_sync with kv_head_major = 0.
 *   Sparse outputs are head-major: k_agg, v_agg dev [Hkv, T, d]; kv_pos dev int32 [Hkv, T] =
 *   off_n + local index; sel_idx_out dev int32 [Hkv, T] local indices (TOPK; nullable);
 *   cu_kv dev int32 [N+1] = prefix sum of k_sel.  Dropped rows are removed, not zeroed.
 *
 *   k_parts, v_parts: host arrays of N dev pointers, participant n's [L_n,Hkv,d] (may be slices
 *   of one packed buffer).  seqlens_host host int32 [N].  k_sel_host host int32 [N], 0 <= k_sel[n]
 *   <= L_n (ignored for CONCAT).  Both TOPK modes need L_n <= 4096 per participant (else
 *   UNSUPPORTED).
 *   kv_pos and cu_kv may be NULL when not wanted. */
typedef enum {
    FEDATTN_AGG_CONCAT = 0,
    FEDATTN_AGG_TOPK_KNORM = 1,
    FEDATTN_AGG_INDEXED = 2,
    FEDATTN_AGG_TOPK_TOKEN = 3
} fedattn_agg_mode;

fedattn_status fedattn_aggregate_kv(fedattn_ctx *ctx, const fedattn_shape *shape, int32_t mode,
                                    const void *const *k_parts, const void *const *v_parts,
                                    const int32_t *seqlens_host, const int32_t *k_sel_host,
                                    const int32_t *sel_idx_in,
                                    void *k_agg, void *v_agg, int32_t *kv_pos, int32_t *cu_kv,
                                    int32_t *sel_idx_out, fedattn_stream stream);

/* ---- global (sync) attention: Phase II, o_n = Attention(q_n, K, V) ----------------------------
 * Paper: Sec. IV-B "Phase II: Global Self-Attention", eq. (update_local_o_H), Algorithm 1 second
 * parallel loop.  The mask is causal on the global token index (so that syncing at every block
 * equals centralised attention): query row i with position p_i = q_pos ? q_pos[i] : i attends
 * aggregated row j of KV head h iff kv_pos[h][j] <= p_i (every row when causal == 0).  A row whose
 * allowed set is empty gets o = 0 and lse = -inf.
 *   q dev [L,Hq,d] (all participants' rows, packed; L = n_q_rows).
 *   k_agg, v_agg dev: kv_head_major == 0: [T,Hkv,d], kv_pos dev int32 [T] or NULL (= 0..T-1);
 *                     kv_head_major == 1: [Hkv,T,d], kv_pos dev int32 [Hkv,T] or NULL.
 *   q_pos dev int32 [L] or NULL.  o dev [L,Hq,d]; lse dev float [L,Hq] or NULL.
 *   Order of positions.  With q_pos == NULL, kv_pos must be non-decreasing along T (what
 *   fedattn_aggregate_kv produces for contiguous segments); the bf16 head_dim 128 kernel then
 *   masks by a prefix count, checks the order as it goes and raises FEDATTN_ERR_ORDER (outputs
 *   undefined) when it does not hold.  With q_pos given, query and key positions may come in ANY
 *   order (general index sets L_n of Sec. IV-A, e.g. interleaved participants; a subset of the
 *   participants' rows): every (query, key) pair is tested on its own positions.  To attend an
 *   unsorted kv_pos from packed queries, pass q_pos = 0..L-1 explicitly. */
fedattn_status fedattn_sync(fedattn_ctx *ctx, const fedattn_shape *shape,
                            const void *q, int64_t n_q_rows, const int32_t *q_pos,
                            const void *k_agg, const void *v_agg, const int32_t *kv_pos,
                            int64_t total_kv, int32_t kv_head_major,
                            void *o, float *lse, fedattn_stream stream);

/* ---- sync block with sparse KV exchange -----------------------------------------------------
 * Paper: Sec. VI, discussion of the sparsity-ratio experiment (the own segment stays complete,
 * only the keys and values received from the other participants are sparsified); Sec. III-B
 * lets the attention operator stand for the masked or the unmasked (bidirectional) form.
 * Row i of participant n attends its own keys (off_n..i when causal, the whole segment otherwise)
 * and the exchanged keys of the OTHER participants that its mask allows, under ONE softmax.  With
 * contiguous segments the second set is "aggregated rows positioned before off_n" (causal) or
 * "aggregated rows positioned outside [off_n, off_{n+1})" (bidirectional), so the block is
 *     fedattn_local (o_a, lse_a)  +  fedattn_sync_remote (o_b, lse_b)  ->  fedattn_merge.
 *
 * fedattn_sync_remote: like fedattn_sync, but query row i of participant n (segments given by the
 *   HOST array cu_seqlens_host [N+1]) attends aggregated row j of KV head h iff
 *   kv_pos[h][j] < off_n, or, when shape->causal == 0, also iff kv_pos[h][j] >= off_{n+1}.
 *   kv_pos must be non-decreasing along T (NULL = 0..T-1).  A row with no such key gets o = 0 and
 *   lse = -inf.  lse is needed for the merge (pass a buffer).
 * fedattn_merge: o = (e^{lse_a} o_a + e^{lse_b} o_b) / (e^{lse_a} + e^{lse_b}),
 *   lse = log(e^{lse_a} + e^{lse_b}) for n_rows query rows; o_a, o_b, o dev [n_rows,Hq,d] in
 *   shape->dtype, lse_a, lse_b dev float [n_rows,Hq], lse dev float or NULL.  o may alias o_a or
 *   o_b.  Two results that are both empty (-inf) merge to o = 0, lse = -inf. */
fedattn_status fedattn_sync_remote(fedattn_ctx *ctx, const fedattn_shape *shape,
                                   const void *q, const int32_t *cu_seqlens_host,
                                   const void *k_agg, const void *v_agg, const int32_t *kv_pos,
                                   int64_t total_kv, int32_t kv_head_major,
                                   void *o, float *lse, fedattn_stream stream);

fedattn_status fedattn_merge(fedattn_ctx *ctx, const fedattn_shape *shape, int64_t n_rows,
                             const void *o_a, const float *lse_a, const void *o_b, const float *lse_b,
                             void *o, float *lse, fedattn_stream stream);

/* ---- decode: one new query token per participant over cached KV -------------------------------
 * Paper: Sec. IV-C "Output Generation" (blocks that ran local attention cache local KV, blocks
 * that ran global attention cache the global KV), Sec. III-C (O(L) per step, memory-bound).
 * The new token is later than every cached row, so no mask applies.
 *   FEDATTN_DECODE_LOCAL  participant n reads rows 0..kv_len[n]-1 of its own cache at
 *                         k_cache + n * cache_stride_participant elements, layout [cap,Hkv,d];
 *                         kv_len dev int32 [N].
 *   FEDATTN_DECODE_SYNC   every participant reads rows 0..kv_len[0]-1 of one shared cache
 *                         [T,Hkv,d]; kv_len dev int32 [1]; cache_stride_participant ignored.
 *   q, o dev [N,Hq,d]; lse dev float [N,Hq] or NULL; max_kv_len >= every kv_len (host; sizes the
 *   split-KV grid).  kv_len = 0 gives o = 0, lse = -inf.  Uses the workspace for split-KV partials.
 *   Two launches per call (stream, then merge), chained by programmatic dependent launch. */
typedef enum { FEDATTN_DECODE_LOCAL = 0, FEDATTN_DECODE_SYNC = 1 } fedattn_decode_mode;

fedattn_status fedattn_decode(fedattn_ctx *ctx, const fedattn_shape *shape, int32_t mode,
                              const void *q, const void *k_cache, const void *v_cache,
                              int64_t cache_stride_participant, const int32_t *kv_len,
                              int32_t max_kv_len, void *o, float *lse, fedattn_stream stream);

/* ---- decode for callers that cannot allocate -------------------------------------------------
 * (The paper has no counterpart; this is a packaging variant of fedattn_decode.)
 * fedattn_decode needs a context whose workspace somebody allocated with cudaMalloc (or a
 * framework allocator).  Some callers cannot do that: code running where the device allocator
 * must not be entered (inside a serving loop with a frozen memory plan, a plugin that receives
 * its tensors and nothing more, a process whose memory is fully pre-partitioned).  This entry
 * point takes no context and allocates nothing, on the host or on the device: the split-KV
 * partials go to a fixed 8.25 MiB array built into the library image, which every GPU that loads
 * the library holds until the process exits.
 *
 * Same arguments, layouts and results as fedattn_decode (bf16, head_dim 128 only; anything else
 * returns FEDATTN_ERR_UNSUPPORTED).  The built-in scratch covers n_participants * n_q_heads <= 256
 * output rows; a larger shape is rejected with FEDATTN_ERR_WORKSPACE and nothing is launched.
 * It runs on the CURRENT device.  The first call on each device resolves the array's device
 * address and sets kernel attributes; make that first call outside any stream capture.  The
 * partial slots need not start at zero (every slot that is read is written earlier in the same
 * call) and their contents after a call are unspecified.  All calls on one device share the
 * array: two calls that may overlap on the GPU (different streams, no ordering) race on it.
 * The first call on a device also fills a small host-side table without locking: do not let two
 * host threads make their first call on the same device at the same moment. */
fedattn_status fedattn_decode_noalloc(const fedattn_shape *shape, int32_t mode,
                                      const void *q, const void *k_cache, const void *v_cache,
                                      int64_t cache_stride_participant, const int32_t *kv_len,
                                      int32_t max_kv_len, void *o, float *lse, fedattn_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* FEDATTN_H_ */
