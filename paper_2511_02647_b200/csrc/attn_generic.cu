// Generic SIMT attention kernel: fp32 or bf16 storage, fp32 arithmetic, head_dim <= 128.
// Serves the fp32 configuration (tensor cores have no fp32 kind and TF32 would miss the 1e-4
// bound), head dims the tensor-core kernel does not cover, explicit query positions, and the
// fp32 decode path.  One warp owns one (query row, query head): lanes split the keys of a
// 32-key block for the logits, and split the head dimension for the weighted value sum.
#include "common.cuh"

namespace fedattn {

template <typename T> __device__ __forceinline__ float ld_f(const T *p);
template <> __device__ __forceinline__ float ld_f<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __bfloat162float(*p);
}
template <typename T> __device__ __forceinline__ void st_f(T *p, float x);
template <> __device__ __forceinline__ void st_f<float>(float *p, float x) { *p = x; }
template <> __device__ __forceinline__ void st_f<__nv_bfloat16>(__nv_bfloat16 *p, float x) {
    *p = __float2bfloat16_rn(x);
}

constexpr int kWarpsPerBlock = 4;

template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
attn_generic_kernel(const GenericParams p)
{
    __shared__ float q_s[kWarpsPerBlock][FEDATTN_MAX_HEAD_DIM];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t item = (int64_t)blockIdx.x * kWarpsPerBlock + warp;
    if (item >= p.n_rows * p.hq) return;            // whole warp leaves together
    const int64_t row = item / p.hq;
    const int h = (int)(item % p.hq);
    const int kvh = h / (p.hq / p.hkv);
    const int d = p.d;

    // Key range and position test for this row.
    int64_t kv_lo = 0, kv_hi = 0;
    int64_t pos = p.q_pos ? p.q_pos[row] : row;
    int64_t kv_base = (int64_t)kvh * p.kv_head_stride;
    bool test_pos = p.causal != 0;
    int64_t own_lo = 0, own_hi = 0;                  // remote-only, bidirectional: positions of the row's own segment
    bool test_own = false;
    if (p.mode == kLocal) {
        int n = 0;
        while (n + 1 < p.n_seg && row >= p.cu[n + 1]) ++n;
        kv_lo = p.cu[n];
        kv_hi = p.causal ? row + 1 : (int64_t)p.cu[n + 1];
        test_pos = false;
    } else if (p.mode == kSync) {
        if (p.remote_only) {
            int n = 0;
            while (n + 1 < p.n_seg && row >= p.cu[n + 1]) ++n;
            if (p.causal) {
                pos = (int64_t)p.cu[n] - 1;          // position = last one before the row's own segment
            } else {                                 // everything positioned outside the row's own segment
                own_lo = p.cu[n]; own_hi = p.cu[n + 1];
                test_own = true;
            }
        }
        kv_hi = p.total_kv;
        if (p.causal && !p.kv_pos) {                 // identity positions: a prefix
            kv_hi = min(kv_hi, pos + 1);
            if (kv_hi < 0) kv_hi = 0;
            test_pos = false;
        }
    } else if (p.mode == kDecodeLocal) {
        kv_hi = p.kv_len[row];
        kv_base += row * p.cache_stride;
        test_pos = false;
    } else {
        kv_hi = p.kv_len[0];
        test_pos = false;
    }
    const T *K = reinterpret_cast<const T *>(p.k) + kv_base;
    const T *V = reinterpret_cast<const T *>(p.v) + kv_base;
    const int32_t *kvp = p.kv_pos ? p.kv_pos + (int64_t)kvh * p.kv_pos_head_stride : nullptr;

    const T *qrow = reinterpret_cast<const T *>(p.q) + (row * p.hq + h) * d;
    for (int c = lane; c < d; c += 32) q_s[warp][c] = ld_f(qrow + c);
    __syncwarp();

    float m = -INFINITY, l = 0.f;
    float acc[FEDATTN_MAX_HEAD_DIM / 32];
#pragma unroll
    for (int i = 0; i < FEDATTN_MAX_HEAD_DIM / 32; ++i) acc[i] = 0.f;

    for (int64_t j0 = kv_lo; j0 < kv_hi; j0 += 32) {
        const int64_t j = j0 + lane;
        bool ok = j < kv_hi;
        if (ok && test_pos) ok = (int64_t)(kvp ? kvp[j] : j) <= pos;
        if (ok && test_own) {
            const int64_t pj = kvp ? kvp[j] : j;
            ok = pj < own_lo || pj >= own_hi;
        }
        float s = -INFINITY;
        if (ok) {
            const T *kr = K + j * p.kv_tok_stride;
            float dot = 0.f;
            for (int c = 0; c < d; ++c) dot = fmaf(q_s[warp][c], ld_f(kr + c), dot);
            s = dot * p.scale;
        }
        float bm = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        if (bm == -INFINITY) continue;               // nothing allowed in this block (uniform)
        const float m_new = fmaxf(m, bm);
        const float alpha = (m == -INFINITY) ? 0.f : expf(m - m_new);
        const float pj = ok ? expf(s - m_new) : 0.f;
        float ps = pj;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        l = l * alpha + ps;
        m = m_new;
#pragma unroll
        for (int i = 0; i < FEDATTN_MAX_HEAD_DIM / 32; ++i) acc[i] *= alpha;
        const int nk = (int)min((int64_t)32, kv_hi - j0);
        for (int t = 0; t < nk; ++t) {
            const float pt = __shfl_sync(0xffffffffu, pj, t);
            if (pt == 0.f) continue;                 // uniform across the warp
            const T *vr = V + (j0 + t) * p.kv_tok_stride;
#pragma unroll
            for (int i = 0; i < FEDATTN_MAX_HEAD_DIM / 32; ++i) {
                const int c = lane + 32 * i;
                if (c < d) acc[i] = fmaf(pt, ld_f(vr + c), acc[i]);
            }
        }
    }
    T *orow = reinterpret_cast<T *>(p.o) + (row * p.hq + h) * d;
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int i = 0; i < FEDATTN_MAX_HEAD_DIM / 32; ++i) {
        const int c = lane + 32 * i;
        if (c < d) st_f(orow + c, acc[i] * inv);
    }
    if (p.lse && lane == 0) p.lse[row * p.hq + h] = l > 0.f ? m + logf(l) : -INFINITY;
}

cudaError_t launch_attn_generic(const GenericParams &p, int dtype, cudaStream_t s, int64_t *launches)
{
    const int64_t items = p.n_rows * p.hq;
    if (items == 0) return cudaSuccess;
    const int64_t blocks = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    if (dtype == FEDATTN_F32)
        attn_generic_kernel<float><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, s>>>(p);
    else
        attn_generic_kernel<__nv_bfloat16><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, s>>>(p);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace fedattn
