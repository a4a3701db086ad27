// KV aggregation kernels: dense concatenation, key-norm scores, per-(participant, head) top-k
// selection, and the indexed gather that builds the head-major sparse KV.  All are pure data
// movement or integer/compare work except the score, which is an fp64 chain in fixed order so
// that the selected set is bit-identical to a sequential fp64 evaluation.
#include "common.cuh"

namespace fedattn {

__device__ __forceinline__ int find_segment(const int32_t *pre, int n, int32_t x)
{
    // largest s in [0, n) with pre[s] <= x, skipping empty segments (pre non-decreasing)
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (pre[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// ---- dense concatenation -----------------------------------------------------------------------
// grid.y = 0 copies K, 1 copies V.  Each thread moves 16-byte vectors; 4 loads are issued before
// the 4 stores so that enough bytes are in flight per SM.
constexpr int kCopyUnroll = 4;

__global__ void __launch_bounds__(256)
concat_kernel(const PartsParams pp, int64_t row_vecs, int64_t total_vecs, uint4 *k_agg, uint4 *v_agg,
              int32_t *kv_pos, int32_t *cu_kv)
{
    const bool is_v = blockIdx.y != 0;
    uint4 *dst = is_v ? v_agg : k_agg;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t base = tid; base < total_vecs; base += stride * kCopyUnroll) {
        uint4 val[kCopyUnroll];
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int64_t i = base + u * stride;
            if (i < total_vecs) {
                const int32_t row = (int32_t)(i / row_vecs);
                const int n = find_segment(pp.off, pp.n, row);
                const uint4 *src = reinterpret_cast<const uint4 *>(is_v ? pp.v[n] : pp.k[n]);
                val[u] = ld_stream(src + (i - (int64_t)pp.off[n] * row_vecs));
            }
        }
#pragma unroll
        for (int u = 0; u < kCopyUnroll; ++u) {
            const int64_t i = base + u * stride;
            if (i < total_vecs) dst[i] = val[u];
        }
    }
    if (!is_v) {
        const int32_t L = pp.off[pp.n];
        if (kv_pos)
            for (int64_t i = tid; i < L; i += stride) kv_pos[i] = (int32_t)i;
        if (cu_kv && tid <= pp.n) cu_kv[tid] = pp.off[tid];
    }
}

cudaError_t launch_concat(const PartsParams &pp, int hkv, int d, int elt_bytes, void *k_agg, void *v_agg,
                          int32_t *kv_pos, int32_t *cu_kv, cudaStream_t s, int sm_count, int64_t *launches)
{
    const int64_t row_vecs = (int64_t)hkv * d * elt_bytes / 16;
    const int64_t total = row_vecs * pp.off[pp.n];
    int64_t blocks = (total + 256 * kCopyUnroll - 1) / (256 * kCopyUnroll);
    const int64_t cap = (int64_t)sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    concat_kernel<<<dim3((unsigned)blocks, 2), 256, 0, s>>>(pp, row_vecs, total, (uint4 *)k_agg, (uint4 *)v_agg,
                                                            kv_pos, cu_kv);
    ++*launches;
    return cudaGetLastError();
}

// ---- key-norm scores -----------------------------------------------------------------------------
// One thread per (token, KV head): s = sum_c x_c^2 accumulated in fp64 in increasing c.  Each
// square of a bf16/fp32 value is exact in fp64, so only the summation order matters and it is
// fixed here.  Output index: Hkv * off[n] + h * L_n + j.
__device__ __forceinline__ double sq_acc_bf16x2(double s, uint32_t w)
{
    const double lo = (double)__uint_as_float(w << 16);
    const double hi = (double)__uint_as_float(w & 0xffff0000u);
    s = __dadd_rn(s, __dmul_rn(lo, lo));
    s = __dadd_rn(s, __dmul_rn(hi, hi));
    return s;
}

template <int kDtype>
__global__ void __launch_bounds__(256)
knorm_score_kernel(const PartsParams pp, int hkv, int d, double *scores)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t total = (int64_t)pp.off[pp.n] * hkv;
    if (t >= total) return;
    const int32_t row = (int32_t)(t / hkv);
    const int h = (int)(t % hkv);
    const int n = find_segment(pp.off, pp.n, row);
    const int32_t j = row - pp.off[n];
    const int32_t len = pp.off[n + 1] - pp.off[n];
    double s = 0.0;
    if (kDtype == FEDATTN_BF16) {
        const uint4 *src = reinterpret_cast<const uint4 *>(
            reinterpret_cast<const __nv_bfloat16 *>(pp.k[n]) + ((int64_t)j * hkv + h) * d);
        for (int c = 0; c < d / 8; ++c) {
            const uint4 w = __ldg(src + c);
            s = sq_acc_bf16x2(s, w.x);
            s = sq_acc_bf16x2(s, w.y);
            s = sq_acc_bf16x2(s, w.z);
            s = sq_acc_bf16x2(s, w.w);
        }
    } else {
        const float4 *src = reinterpret_cast<const float4 *>(
            reinterpret_cast<const float *>(pp.k[n]) + ((int64_t)j * hkv + h) * d);
        for (int c = 0; c < d / 4; ++c) {
            const float4 w = __ldg(src + c);
            s = __dadd_rn(s, __dmul_rn((double)w.x, (double)w.x));
            s = __dadd_rn(s, __dmul_rn((double)w.y, (double)w.y));
            s = __dadd_rn(s, __dmul_rn((double)w.z, (double)w.z));
            s = __dadd_rn(s, __dmul_rn((double)w.w, (double)w.w));
        }
    }
    scores[(int64_t)hkv * pp.off[n] + (int64_t)h * len + j] = s;
}

cudaError_t launch_knorm_scores(const PartsParams &pp, int hkv, int d, int dtype, double *scores,
                                cudaStream_t s, int64_t *launches)
{
    const int64_t total = (int64_t)pp.off[pp.n] * hkv;
    if (total == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (dtype == FEDATTN_BF16)
        knorm_score_kernel<FEDATTN_BF16><<<blocks, 256, 0, s>>>(pp, hkv, d, scores);
    else
        knorm_score_kernel<FEDATTN_F32><<<blocks, 256, 0, s>>>(pp, hkv, d, scores);
    ++*launches;
    return cudaGetLastError();
}

// ---- top-k selection ---------------------------------------------------------------------------
// One CTA per (KV head, participant).  Scores are non-negative doubles, so their bit patterns
// order like unsigned integers.  An 8-bit-per-pass radix select finds the k-th largest score
// tau and how many rows equal to tau are still needed; an ordered compaction then emits, in
// ascending index order, every row with score > tau plus the lowest-index rows with score == tau.
constexpr int kSelThreads = 256;
constexpr int kSelMaxLen = 4096;

__device__ __forceinline__ int block_excl_scan_flag(bool flag, int *warp_tot, int &block_total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned bal = __ballot_sync(0xffffffffu, flag);
    const int in_warp = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) {
        const int c = warp_tot[w];
        if (w < warp) base += c;
        tot += c;
    }
    __syncthreads();
    block_total = tot;
    return base + in_warp;
}

__global__ void __launch_bounds__(kSelThreads)
topk_select_kernel(const PartsParams pp, int hkv, const double *scores, int32_t *sel_idx)
{
    __shared__ unsigned long long keys[kSelMaxLen];
    __shared__ int hist[256];
    __shared__ int warp_tot[kSelThreads / 32];
    __shared__ int sh_bin, sh_krem;

    const int h = blockIdx.x, n = blockIdx.y;
    const int len = pp.off[n + 1] - pp.off[n];
    const int k = pp.cu_kv[n + 1] - pp.cu_kv[n];
    if (k == 0 || len == 0) return;
    const int64_t T = pp.cu_kv[pp.n];
    const double *sc = scores + (int64_t)hkv * pp.off[n] + (int64_t)h * len;
    for (int j = threadIdx.x; j < len; j += kSelThreads)
        keys[j] = (unsigned long long)__double_as_longlong(sc[j]);
    __syncthreads();

    unsigned long long prefix = 0, mask = 0;
    int k_rem = k;
    for (int shift = 56; shift >= 0; shift -= 8) {
        hist[threadIdx.x] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < len; j += kSelThreads) {
            const unsigned long long key = keys[j];
            if ((key & mask) == prefix) atomicAdd(&hist[(int)((key >> shift) & 0xff)], 1);
        }
        __syncthreads();
        // suffix sums over bins: S[b] = sum_{b' >= b} hist[b']
        const int b = threadIdx.x;
        const int mine = hist[b];
        const int lane = b & 31, warp = b >> 5;
        int incl = mine;   // inclusive suffix within warp: sum over lanes >= lane
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_down_sync(0xffffffffu, incl, o);
            if (lane + o < 32) incl += up;
        }
        if (lane == 0) warp_tot[warp] = incl;
        __syncthreads();
        int above = 0;
#pragma unroll
        for (int w = 0; w < kSelThreads / 32; ++w)
            if (w > warp) above += warp_tot[w];
        const int S_b = incl + above;       // count of candidates with byte >= b
        const int S_next = S_b - mine;      // count with byte > b
        if (S_b >= k_rem && S_next < k_rem) {
            sh_bin = b;
            sh_krem = k_rem - S_next;
        }
        __syncthreads();
        prefix |= (unsigned long long)sh_bin << shift;
        mask |= 0xffULL << shift;
        k_rem = sh_krem;
        __syncthreads();
    }
    const unsigned long long tau = prefix;   // k-th largest score; k_rem rows equal to tau are kept

    int eq_base = 0, out_base = 0;
    int32_t *dst = sel_idx + (int64_t)h * T + pp.cu_kv[n];
    for (int j0 = 0; j0 < len; j0 += kSelThreads) {
        const int j = j0 + threadIdx.x;
        const unsigned long long key = j < len ? keys[j] : 0ULL;
        const bool is_eq = j < len && key == tau;
        int eq_tot, sel_tot;
        const int eq_rank = eq_base + block_excl_scan_flag(is_eq, warp_tot, eq_tot);
        const bool sel = j < len && (key > tau || (is_eq && eq_rank < k_rem));
        const int pos = out_base + block_excl_scan_flag(sel, warp_tot, sel_tot);
        if (sel) dst[pos] = j;
        eq_base += eq_tot;
        out_base += sel_tot;
    }
}

cudaError_t launch_topk_select(const PartsParams &pp, int hkv, const double *scores, int32_t *sel_idx,
                               cudaStream_t s, int64_t *launches)
{
    if (pp.cu_kv[pp.n] == 0) return cudaSuccess;
    topk_select_kernel<<<dim3(hkv, pp.n), kSelThreads, 0, s>>>(pp, hkv, scores, sel_idx);
    ++*launches;
    return cudaGetLastError();
}

// ---- indexed gather ------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gather_kernel(const PartsParams pp, int hkv, int64_t vpr /* 16-byte vectors per (row, head) */,
              const int32_t *sel_idx, uint4 *k_agg, uint4 *v_agg, int32_t *kv_pos, int32_t *cu_kv,
              int32_t *sel_idx_out, int32_t *status)
{
    const int64_t T = pp.cu_kv[pp.n];
    const int64_t total = (int64_t)hkv * T * vpr;
    const bool is_v = blockIdx.y != 0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = tid; i < total; i += stride) {
        const int64_t rowid = i / vpr;               // h * T + t
        const int vi = (int)(i - rowid * vpr);
        const int h = (int)(rowid / T);
        const int32_t t = (int32_t)(rowid - (int64_t)h * T);
        const int n = find_segment(pp.cu_kv, pp.n, t);
        const int32_t j = sel_idx[rowid];
        const int32_t len = pp.off[n + 1] - pp.off[n];
        if (j < 0 || j >= len) {
            if (vi == 0) atomicMax(status, (int32_t)FEDATTN_ERR_INDEX);
            continue;
        }
        const uint4 *src = reinterpret_cast<const uint4 *>(is_v ? pp.v[n] : pp.k[n]) +
                           ((int64_t)j * hkv + h) * vpr + vi;
        (is_v ? v_agg : k_agg)[i] = ld_stream(src);
        if (vi == 0 && !is_v) {
            if (kv_pos) kv_pos[rowid] = pp.off[n] + j;
            if (sel_idx_out && sel_idx_out != sel_idx) sel_idx_out[rowid] = j;
        }
    }
    if (!is_v && cu_kv && tid <= pp.n) cu_kv[tid] = pp.cu_kv[tid];
}

cudaError_t launch_gather(const PartsParams &pp, int hkv, int d, int elt_bytes, const int32_t *sel_idx,
                          void *k_agg, void *v_agg, int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out,
                          int32_t *status, cudaStream_t s, int64_t *launches)
{
    const int64_t vpr = (int64_t)d * elt_bytes / 16;
    const int64_t total = (int64_t)hkv * pp.cu_kv[pp.n] * vpr;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    gather_kernel<<<dim3((unsigned)blocks, 2), 256, 0, s>>>(pp, hkv, vpr, sel_idx, (uint4 *)k_agg, (uint4 *)v_agg,
                                                            kv_pos, cu_kv, sel_idx_out, status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace fedattn
