// Shared declarations of the FedAttn CUDA library (host dispatch <-> kernel launchers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fedattn.h"

namespace fedattn {

// Workspace layout: [0, 256) status area (word 0: the status word; bytes 64..71: the sequence number of the
// latest sparse aggregation known to be complete), then the scratch region.
constexpr size_t kStatusBytes = 256;
constexpr size_t kDoneSeqOffset = 64;
constexpr int kMaxP = FEDATTN_MAX_PARTICIPANTS;
// Upper bound on spin iterations of any in-kernel wait before it gives up.
constexpr uint32_t kSpinLimit = 1u << 22;

struct Context {
    int device;
    int sm_count;
    char *workspace;       // dev
    size_t workspace_bytes;
    int32_t *status;       // dev, == workspace
    char *scratch;         // dev, workspace + kStatusBytes
    size_t scratch_bytes;
    int64_t launches;
    int64_t tc_launches;   // launches of the tcgen05 attention kernel among them
    int64_t agg_seq;       // sequence number of the latest sparse aggregation call
    uint64_t agg_key;      // key of the stream that call ran on (early-start bookkeeping)
    void *encode_tiled;    // cuTensorMapEncodeTiled entry point (driver), or nullptr
};

// ---- early-start bookkeeping (programmatic dependent launch) ------------------------------------
struct MemRange {
    const void *p;
    size_t bytes;
};
struct EarlyStart {
    bool early;          // the inputs may be read before the preceding grid of the stream is complete
    int64_t seq;         // this call's sequence number in its context (0: none, publish nothing)
    int64_t need_seq;    // the context's latest recorded call that reads or writes one of `out` (0: none;
                         // INT64_MAX: one that cannot be named, wait before the first write)
};
// Records `in` (read) and `out` (written) as buffers that grids of this call may still be using when
// later grids of `stream` start, and decides how the call may start.  writes_before_wait: the call's
// kernel writes `out` before its griddepcontrol.wait when need_seq allows it (otherwise overlaps of
// `out` with recorded buffers do not matter).  owner / seq_counter / owner_key: the context's done
// word, its sequence counter and the key of the stream its numbered calls last ran on (all null for
// calls without sequence numbers).
EarlyStart early_start(int device, cudaStream_t stream, const MemRange *in, int n_in, const MemRange *out, int n_out,
                       bool writes_before_wait = false, const void *owner = nullptr, int64_t *seq_counter = nullptr,
                       uint64_t *owner_key = nullptr);
// The owner's sequence numbers are about to lose their meaning (its context is being destroyed).
void early_start_forget(int device, const void *owner);

// ---- generic SIMT attention (fp32 or bf16 storage, any head_dim <= 128) --------------------
enum GenericMode { kLocal = 0, kSync = 1, kDecodeLocal = 2, kDecodeSync = 3 };

struct GenericParams {
    const void *q, *k, *v;
    void *o;
    float *lse;
    int64_t n_rows;               // query rows (tokens, or participants for decode)
    int32_t hq, hkv, d;
    float scale;
    int32_t causal;
    int32_t mode;                 // GenericMode
    int32_t remote_only;          // kSync: a row sees the keys positioned before its segment (cu) and, when
                                  // causal == 0, those positioned after it
    int64_t kv_tok_stride;        // elements between consecutive KV rows of one head
    int64_t kv_head_stride;       // elements between KV heads
    int64_t kv_pos_head_stride;   // ints between heads in kv_pos (0 = shared)
    int64_t total_kv;             // sync: rows of the aggregated KV
    const int32_t *q_pos;         // nullable
    const int32_t *kv_pos;        // nullable
    const int32_t *kv_len;        // decode: dev lengths
    int64_t cache_stride;         // decode local: elements between participants' caches
    int32_t n_seg;
    int32_t cu[kMaxP + 1];        // local: segment offsets
};

cudaError_t launch_attn_generic(const GenericParams &p, int dtype, cudaStream_t s, int64_t *launches);

// ---- aggregation -----------------------------------------------------------------------------
struct PartsParams {
    const void *k[kMaxP];
    const void *v[kMaxP];
    int32_t n;
    int32_t off[kMaxP + 1];       // prefix sum of L_n  (rows)
    int32_t cu_kv[kMaxP + 1];     // prefix sum of k_sel (rows), sparse modes
};

cudaError_t launch_concat(const PartsParams &pp, int hkv, int d, int elt_bytes, void *k_agg, void *v_agg,
                          int32_t *kv_pos, int32_t *cu_kv, cudaStream_t s, int sm_count, int64_t *launches);

cudaError_t launch_topk_fused(const PartsParams &pp, int hkv, int d, int dtype, void *k_agg, void *v_agg,
                              int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out, Context *ctx, cudaStream_t s);
cudaError_t launch_gather(const PartsParams &pp, int hkv, int d, int elt_bytes, const int32_t *sel_idx,
                          void *k_agg, void *v_agg, int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out,
                          int32_t *status, int device, int sm_count, cudaStream_t s, int64_t *launches);

// ---- bf16 prefill on tensor cores (tcgen05 + TMEM + TMA), head_dim 128 ------------------------
struct PrefillParams {
    const void *q, *k, *v;
    void *o;
    float *lse;
    int64_t n_q_rows;
    int64_t total_kv;             // rows of K/V (== n_q_rows for local)
    int32_t hq, hkv;
    float scale;
    int32_t causal;
    int32_t sync;                 // 0 local, 1 sync
    int32_t remote_only;          // sync: a row sees the aggregated rows positioned before its segment (and, when
                                  // causal == 0, those positioned after it)
    int32_t kv_head_major;
    const int32_t *kv_pos;        // nullable
    int32_t general;              // sync, causal: every (query, key) pair is tested on explicit positions
    const int32_t *q_pos;         // general: nullable (= row index)
    int32_t *tab;                 // general: scratch for the position tables (position_table_bytes)
    int32_t n_seg;
    int32_t cu[kMaxP + 1];        // query segments (local: also the KV segments)
};
bool prefill_sm100_supported(const Context *ctx);
// scratch bytes of the per-tile position tables of a general-position sync call
size_t position_table_bytes(int hkv, int64_t n_q_rows, int64_t total_kv);
cudaError_t launch_prefill_sm100(Context *ctx, const PrefillParams &p, cudaStream_t s);
// one small kernel whose bounded wait runs out after max_polls polls (raises FEDATTN_ERR_TIMEOUT)
cudaError_t launch_wait_selftest(Context *ctx, int max_polls, cudaStream_t s);

// ---- merge of two partial attention results through their log-sum-exps ----------------------
cudaError_t launch_merge(int dtype, int64_t n_rows, int hq, int d, const void *o_a, const float *lse_a, const void *o_b,
                         const float *lse_b, void *o, float *lse, int sm_count, cudaStream_t s, int64_t *launches);

// ---- bf16 split-KV decode (tensor-core scores, warp-shuffle softmax) ---------------------------
struct DecodeParams {
    const void *q, *k, *v;
    void *o;
    float *lse;
    int32_t n_part, hq, hkv, d;
    float scale;
    int32_t sync;
    int64_t cache_stride;
    const int32_t *kv_len;
    int32_t max_kv_len;
    float *partial;               // scratch: per-split partial results
    size_t partial_bytes;
    int32_t g_shift;              // log2(hq / hkv) when that is a power of two, else -1 (set by the launcher)
    int32_t early;                // inputs may be read before the preceding grid is complete (set by the launcher)
};
size_t decode_scratch_bytes(int n_part, int hq, int d, int sm_count);
cudaError_t launch_decode_bf16(const Context *ctx, const DecodeParams &p, cudaStream_t s, int64_t *launches);

}  // namespace fedattn
