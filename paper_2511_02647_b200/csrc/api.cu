// Host side of the C ABI: context, argument validation, dispatch.  No arithmetic of the method
// happens here; every step runs in the kernels this file launches.
#include <math.h>
#include <new>
#include <string.h>

#include "common.cuh"

using namespace fedattn;

struct fedattn_ctx {
    Context c;
};

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool shape_ok(const fedattn_shape *s)
{
    if (!s) return false;
    if (s->n_participants < 1 || s->n_participants > FEDATTN_MAX_PARTICIPANTS) return false;
    if (s->n_q_heads < 1 || s->n_kv_heads < 1 || s->n_q_heads % s->n_kv_heads != 0) return false;
    if (s->head_dim < 8 || s->head_dim > FEDATTN_MAX_HEAD_DIM || s->head_dim % 8 != 0) return false;
    if (s->dtype != FEDATTN_F32 && s->dtype != FEDATTN_BF16) return false;
    if (s->causal != 0 && s->causal != 1) return false;
    if (!(s->scale >= 0.f) || isinf(s->scale)) return false;
    return true;
}

inline float eff_scale(const fedattn_shape *s)
{
    return s->scale > 0.f ? s->scale : 1.0f / sqrtf((float)s->head_dim);
}

inline int elt_bytes(const fedattn_shape *s) { return s->dtype == FEDATTN_BF16 ? 2 : 4; }

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

const char *fedattn_status_string(fedattn_status s)
{
    switch (s) {
    case FEDATTN_OK: return "ok";
    case FEDATTN_ERR_INVALID_ARG: return "invalid argument";
    case FEDATTN_ERR_UNSUPPORTED: return "unsupported configuration";
    case FEDATTN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FEDATTN_ERR_CUDA: return "CUDA call failed";
    case FEDATTN_ERR_TIMEOUT: return "a bounded in-kernel wait ran out";
    case FEDATTN_ERR_INDEX: return "selection index out of range or not ascending";
    case FEDATTN_ERR_ORDER: return "key positions not in non-decreasing order";
    }
    return "unknown status";
}

size_t fedattn_workspace_bytes(const fedattn_shape *shape, int64_t max_total_tokens, int64_t max_total_kv)
{
    if (!shape_ok(shape) || max_total_tokens < 0 || max_total_kv < 0) return 0;
    // scratch, shared by calls that are ordered on one stream: the split-KV partials of the decode
    // kernel, or the position tables of a sync call with explicit query positions
    size_t need = decode_scratch_bytes(shape->n_participants, shape->n_q_heads, shape->head_dim, 0);
    const size_t tab = position_table_bytes(shape->n_kv_heads, max_total_tokens, max_total_kv);
    if (tab > need) need = tab;
    return kStatusBytes + align_up(need, 256);
}

fedattn_status fedattn_create(fedattn_ctx **out, int device, void *workspace, size_t workspace_bytes)
{
    if (!out) return FEDATTN_ERR_INVALID_ARG;
    *out = nullptr;
    if (!workspace || workspace_bytes < kStatusBytes || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return FEDATTN_ERR_WORKSPACE;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return FEDATTN_ERR_CUDA;
    DeviceGuard g(device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FEDATTN_ERR_CUDA;
    fedattn_ctx *ctx = new (std::nothrow) fedattn_ctx();
    if (!ctx) return FEDATTN_ERR_CUDA;
    Context &c = ctx->c;
    c.device = device;
    c.sm_count = prop.multiProcessorCount;
    c.workspace = static_cast<char *>(workspace);
    c.workspace_bytes = workspace_bytes;
    c.status = reinterpret_cast<int32_t *>(workspace);
    c.scratch = c.workspace + kStatusBytes;
    c.scratch_bytes = workspace_bytes - kStatusBytes;
    c.launches = 0;
    c.tc_launches = 0;
    c.agg_seq = 0;
    c.agg_key = ~0ull;
    c.encode_tiled = nullptr;
    if (prop.major == 10) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            c.encode_tiled = fn;
    }
    if (cudaMemset(workspace, 0, kStatusBytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        delete ctx;
        return FEDATTN_ERR_CUDA;
    }
    *out = ctx;
    return FEDATTN_OK;
}

void fedattn_destroy(fedattn_ctx *ctx)
{
    if (ctx) early_start_forget(ctx->c.device, ctx->c.workspace + kDoneSeqOffset);
    delete ctx;
}

int64_t fedattn_launch_count(const fedattn_ctx *ctx) { return ctx ? ctx->c.launches : 0; }

int64_t fedattn_tensor_core_launch_count(const fedattn_ctx *ctx) { return ctx ? ctx->c.tc_launches : 0; }

fedattn_status fedattn_selftest_wait_timeout(fedattn_ctx *ctx, int32_t max_polls, fedattn_stream stream)
{
    if (!ctx || max_polls < 1 || max_polls > 65536) return FEDATTN_ERR_INVALID_ARG;
    if (!prefill_sm100_supported(&ctx->c)) return FEDATTN_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    return launch_wait_selftest(&ctx->c, max_polls, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FEDATTN_OK
                                                                                                       : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_poll(fedattn_ctx *ctx, fedattn_stream stream)
{
    if (!ctx) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FEDATTN_ERR_CUDA;
    if (cudaMemcpy(&word, ctx->c.status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess)
        return FEDATTN_ERR_CUDA;
    if (word != 0 && cudaMemset(ctx->c.status, 0, sizeof(word)) != cudaSuccess) return FEDATTN_ERR_CUDA;
    return static_cast<fedattn_status>(word);
}

fedattn_status fedattn_local(fedattn_ctx *ctx, const fedattn_shape *shape, const void *q, const void *k,
                             const void *v, const int32_t *cu, void *o, float *lse, fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape) || !cu) return FEDATTN_ERR_INVALID_ARG;
    const int N = shape->n_participants;
    if (cu[0] != 0) return FEDATTN_ERR_INVALID_ARG;
    for (int n = 0; n < N; ++n)
        if (cu[n + 1] < cu[n]) return FEDATTN_ERR_INVALID_ARG;
    const int64_t L = cu[N];
    if (L == 0) return FEDATTN_OK;
    if (!q || !k || !v || !o) return FEDATTN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err;
    if (shape->dtype == FEDATTN_BF16 && shape->head_dim == 128 && prefill_sm100_supported(&ctx->c)) {
        PrefillParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k; p.v = v; p.o = o; p.lse = lse;
        p.n_q_rows = L; p.total_kv = L;
        p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.sync = 0; p.kv_head_major = 0;
        p.kv_pos = nullptr; p.n_seg = N;
        memcpy(p.cu, cu, sizeof(int32_t) * (N + 1));
        err = launch_prefill_sm100(&ctx->c, p, s);
    } else {
        GenericParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k; p.v = v; p.o = o; p.lse = lse;
        p.n_rows = L; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = shape->head_dim;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.mode = kLocal;
        p.kv_tok_stride = (int64_t)shape->n_kv_heads * shape->head_dim;
        p.kv_head_stride = shape->head_dim;
        p.n_seg = N;
        memcpy(p.cu, cu, sizeof(int32_t) * (N + 1));
        err = launch_attn_generic(p, shape->dtype, s, &ctx->c.launches);
    }
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_aggregate_kv(fedattn_ctx *ctx, const fedattn_shape *shape, int32_t mode,
                                    const void *const *k_parts, const void *const *v_parts,
                                    const int32_t *seqlens, const int32_t *k_sel, const int32_t *sel_idx_in,
                                    void *k_agg, void *v_agg, int32_t *kv_pos, int32_t *cu_kv,
                                    int32_t *sel_idx_out, fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape) || !k_parts || !v_parts || !seqlens) return FEDATTN_ERR_INVALID_ARG;
    if (mode != FEDATTN_AGG_CONCAT && mode != FEDATTN_AGG_TOPK_KNORM && mode != FEDATTN_AGG_INDEXED &&
        mode != FEDATTN_AGG_TOPK_TOKEN)
        return FEDATTN_ERR_INVALID_ARG;
    const int N = shape->n_participants;
    PartsParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.n = N;
    int64_t L = 0, T = 0;
    for (int n = 0; n < N; ++n) {
        if (seqlens[n] < 0) return FEDATTN_ERR_INVALID_ARG;
        if (seqlens[n] > 0 && (!k_parts[n] || !v_parts[n] || !aligned16(k_parts[n]) || !aligned16(v_parts[n])))
            return FEDATTN_ERR_INVALID_ARG;
        pp.k[n] = k_parts[n];
        pp.v[n] = v_parts[n];
        L += seqlens[n];
        if (L > 0x7fffffffLL) return FEDATTN_ERR_INVALID_ARG;
        pp.off[n + 1] = (int32_t)L;
        if (mode != FEDATTN_AGG_CONCAT) {
            if (!k_sel || k_sel[n] < 0 || k_sel[n] > seqlens[n]) return FEDATTN_ERR_INVALID_ARG;
            T += k_sel[n];
        }
        pp.cu_kv[n + 1] = (int32_t)T;
    }
    if (mode == FEDATTN_AGG_INDEXED && T > 0 && !sel_idx_in) return FEDATTN_ERR_INVALID_ARG;
    const int64_t out_rows = mode == FEDATTN_AGG_CONCAT ? L : T;
    if (out_rows > 0 && (!k_agg || !v_agg || !aligned16(k_agg) || !aligned16(v_agg))) return FEDATTN_ERR_INVALID_ARG;
    if (mode == FEDATTN_AGG_TOPK_KNORM || mode == FEDATTN_AGG_TOPK_TOKEN)
        for (int n = 0; n < N; ++n)
            if (seqlens[n] > 4096) return FEDATTN_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int hkv = shape->n_kv_heads, d = shape->head_dim, eb = elt_bytes(shape);
    cudaError_t err = cudaSuccess;
    if (mode == FEDATTN_AGG_CONCAT) {
        err = launch_concat(pp, hkv, d, eb, k_agg, v_agg, kv_pos, cu_kv, s, ctx->c.sm_count, &ctx->c.launches);
        return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
    }
    if (mode == FEDATTN_AGG_TOPK_KNORM) {
        err = launch_topk_fused(pp, hkv, d, shape->dtype, k_agg, v_agg, kv_pos, cu_kv, sel_idx_out, &ctx->c, s);
        return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
    }
    if (mode == FEDATTN_AGG_TOPK_TOKEN) {
        // the per-head kernel on the token row viewed as one head of Hkv * d channels: token-major output
        err = launch_topk_fused(pp, 1, hkv * d, shape->dtype, k_agg, v_agg, kv_pos, cu_kv, sel_idx_out, &ctx->c, s);
        return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
    }
    const int32_t *sel = sel_idx_in;
    err = launch_gather(pp, hkv, d, eb, sel, k_agg, v_agg, kv_pos, cu_kv, sel_idx_out, ctx->c.status, ctx->c.device, ctx->c.sm_count, s,
                        &ctx->c.launches);
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_sync(fedattn_ctx *ctx, const fedattn_shape *shape, const void *q, int64_t n_q_rows,
                            const int32_t *q_pos, const void *k_agg, const void *v_agg, const int32_t *kv_pos,
                            int64_t total_kv, int32_t kv_head_major, void *o, float *lse, fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape) || n_q_rows < 0 || total_kv < 0) return FEDATTN_ERR_INVALID_ARG;
    if (n_q_rows > 0x7fffffffLL || total_kv > 0x7fffffffLL) return FEDATTN_ERR_INVALID_ARG;
    if (kv_head_major != 0 && kv_head_major != 1) return FEDATTN_ERR_INVALID_ARG;
    if (n_q_rows == 0) return FEDATTN_OK;
    if (!q || !o || !aligned16(q) || !aligned16(o)) return FEDATTN_ERR_INVALID_ARG;
    if (total_kv > 0 && (!k_agg || !v_agg || !aligned16(k_agg) || !aligned16(v_agg))) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err;
    if (shape->dtype == FEDATTN_BF16 && shape->head_dim == 128 && total_kv > 0 && prefill_sm100_supported(&ctx->c)) {
        PrefillParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_agg; p.v = v_agg; p.o = o; p.lse = lse;
        p.n_q_rows = n_q_rows; p.total_kv = total_kv;
        p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.sync = 1; p.kv_head_major = kv_head_major;
        p.kv_pos = kv_pos; p.n_seg = 1;
        if (q_pos && shape->causal) {
            // explicit query positions: every (query, key) pair is tested on its own positions, in any order
            if (ctx->c.scratch_bytes < position_table_bytes(p.hkv, n_q_rows, total_kv)) return FEDATTN_ERR_WORKSPACE;
            p.general = 1; p.q_pos = q_pos;
            p.tab = reinterpret_cast<int32_t *>(ctx->c.scratch);
        }
        p.cu[0] = 0; p.cu[1] = (int32_t)n_q_rows;
        err = launch_prefill_sm100(&ctx->c, p, s);
    } else {
        GenericParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_agg; p.v = v_agg; p.o = o; p.lse = lse;
        p.n_rows = n_q_rows; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = shape->head_dim;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.mode = kSync;
        if (kv_head_major) {
            p.kv_tok_stride = shape->head_dim;
            p.kv_head_stride = total_kv * shape->head_dim;
            p.kv_pos_head_stride = total_kv;
        } else {
            p.kv_tok_stride = (int64_t)shape->n_kv_heads * shape->head_dim;
            p.kv_head_stride = shape->head_dim;
            p.kv_pos_head_stride = 0;
        }
        p.total_kv = total_kv; p.q_pos = q_pos; p.kv_pos = kv_pos;
        err = launch_attn_generic(p, shape->dtype, s, &ctx->c.launches);
    }
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_sync_remote(fedattn_ctx *ctx, const fedattn_shape *shape, const void *q, const int32_t *cu,
                                   const void *k_agg, const void *v_agg, const int32_t *kv_pos, int64_t total_kv,
                                   int32_t kv_head_major, void *o, float *lse, fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape) || !cu || total_kv < 0 || total_kv > 0x7fffffffLL) return FEDATTN_ERR_INVALID_ARG;
    if (kv_head_major != 0 && kv_head_major != 1) return FEDATTN_ERR_INVALID_ARG;
    const int N = shape->n_participants;
    if (cu[0] != 0) return FEDATTN_ERR_INVALID_ARG;
    for (int n = 0; n < N; ++n)
        if (cu[n + 1] < cu[n]) return FEDATTN_ERR_INVALID_ARG;
    const int64_t L = cu[N];
    if (L == 0) return FEDATTN_OK;
    if (!q || !o || !aligned16(q) || !aligned16(o)) return FEDATTN_ERR_INVALID_ARG;
    if (total_kv > 0 && (!k_agg || !v_agg || !aligned16(k_agg) || !aligned16(v_agg))) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err;
    if (shape->dtype == FEDATTN_BF16 && shape->head_dim == 128 && total_kv > 0 && prefill_sm100_supported(&ctx->c)) {
        PrefillParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_agg; p.v = v_agg; p.o = o; p.lse = lse;
        p.n_q_rows = L; p.total_kv = total_kv;
        p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.sync = 1; p.remote_only = 1; p.kv_head_major = kv_head_major;
        p.kv_pos = kv_pos; p.n_seg = N;
        memcpy(p.cu, cu, sizeof(int32_t) * (N + 1));
        err = launch_prefill_sm100(&ctx->c, p, s);
    } else {
        GenericParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_agg; p.v = v_agg; p.o = o; p.lse = lse;
        p.n_rows = L; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = shape->head_dim;
        p.scale = eff_scale(shape); p.causal = shape->causal; p.mode = kSync; p.remote_only = 1;
        if (kv_head_major) {
            p.kv_tok_stride = shape->head_dim;
            p.kv_head_stride = total_kv * shape->head_dim;
            p.kv_pos_head_stride = total_kv;
        } else {
            p.kv_tok_stride = (int64_t)shape->n_kv_heads * shape->head_dim;
            p.kv_head_stride = shape->head_dim;
            p.kv_pos_head_stride = 0;
        }
        p.total_kv = total_kv; p.kv_pos = kv_pos;
        p.n_seg = N;
        memcpy(p.cu, cu, sizeof(int32_t) * (N + 1));
        err = launch_attn_generic(p, shape->dtype, s, &ctx->c.launches);
    }
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_merge(fedattn_ctx *ctx, const fedattn_shape *shape, int64_t n_rows, const void *o_a,
                             const float *lse_a, const void *o_b, const float *lse_b, void *o, float *lse,
                             fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape) || n_rows < 0) return FEDATTN_ERR_INVALID_ARG;
    if (n_rows == 0) return FEDATTN_OK;
    if (!o_a || !o_b || !lse_a || !lse_b || !o) return FEDATTN_ERR_INVALID_ARG;
    if (!aligned16(o_a) || !aligned16(o_b) || !aligned16(o)) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaError_t err = launch_merge(shape->dtype, n_rows, shape->n_q_heads, shape->head_dim, o_a, lse_a, o_b, lse_b, o, lse,
                                   ctx->c.sm_count, static_cast<cudaStream_t>(stream), &ctx->c.launches);
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

fedattn_status fedattn_decode(fedattn_ctx *ctx, const fedattn_shape *shape, int32_t mode, const void *q,
                              const void *k_cache, const void *v_cache, int64_t cache_stride,
                              const int32_t *kv_len, int32_t max_kv_len, void *o, float *lse,
                              fedattn_stream stream)
{
    if (!ctx || !shape_ok(shape)) return FEDATTN_ERR_INVALID_ARG;
    if (mode != FEDATTN_DECODE_LOCAL && mode != FEDATTN_DECODE_SYNC) return FEDATTN_ERR_INVALID_ARG;
    if (!q || !o || !kv_len || max_kv_len < 0 || cache_stride < 0) return FEDATTN_ERR_INVALID_ARG;
    if (max_kv_len > 0 && (!k_cache || !v_cache || !aligned16(k_cache) || !aligned16(v_cache)))
        return FEDATTN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(o)) return FEDATTN_ERR_INVALID_ARG;
    if (mode == FEDATTN_DECODE_LOCAL && (cache_stride * elt_bytes(shape)) % 16 != 0) return FEDATTN_ERR_INVALID_ARG;
    DeviceGuard g(ctx->c.device);
    if (!g.ok) return FEDATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err;
    const int N = shape->n_participants;
    const size_t need = decode_scratch_bytes(N, shape->n_q_heads, shape->head_dim, ctx->c.sm_count);
    if (shape->dtype == FEDATTN_BF16 && shape->head_dim == 128 && need > 0) {
        if (ctx->c.scratch_bytes < need) return FEDATTN_ERR_WORKSPACE;
        DecodeParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_cache; p.v = v_cache; p.o = o; p.lse = lse;
        p.n_part = N; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = shape->head_dim;
        p.scale = eff_scale(shape); p.sync = mode == FEDATTN_DECODE_SYNC;
        p.cache_stride = cache_stride; p.kv_len = kv_len; p.max_kv_len = max_kv_len;
        p.partial = reinterpret_cast<float *>(ctx->c.scratch); p.partial_bytes = ctx->c.scratch_bytes;
        err = launch_decode_bf16(&ctx->c, p, s, &ctx->c.launches);
    } else {
        GenericParams p;
        memset(&p, 0, sizeof(p));
        p.q = q; p.k = k_cache; p.v = v_cache; p.o = o; p.lse = lse;
        p.n_rows = N; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = shape->head_dim;
        p.scale = eff_scale(shape); p.causal = 0;
        p.mode = mode == FEDATTN_DECODE_SYNC ? kDecodeSync : kDecodeLocal;
        p.kv_tok_stride = (int64_t)shape->n_kv_heads * shape->head_dim;
        p.kv_head_stride = shape->head_dim;
        p.kv_len = kv_len; p.cache_stride = cache_stride;
        err = launch_attn_generic(p, shape->dtype, s, &ctx->c.launches);
    }
    return err == cudaSuccess ? FEDATTN_OK : FEDATTN_ERR_CUDA;
}

}  // extern "C"
