// Merge of two partial attention results over disjoint key sets A and B of the same queries:
//   o = (e^{lse_a} o_a + e^{lse_b} o_b) / (e^{lse_a} + e^{lse_b}),   lse = log(e^{lse_a} + e^{lse_b}).
// Used for the sync block with sparse KV exchange: A = the participant's own complete segment
// (fedattn_local), B = the exchanged keys of earlier participants (fedattn_sync_remote).
// Pure streaming: every thread owns 8 consecutive channels of one (row, head).
#include "common.cuh"

namespace fedattn {

template <typename T> struct Vec8;
template <> struct Vec8<__nv_bfloat16> {
    uint4 raw;
    __device__ void load(const __nv_bfloat16 *p) { raw = *reinterpret_cast<const uint4 *>(p); }
    __device__ void store(__nv_bfloat16 *p) const { *reinterpret_cast<uint4 *>(p) = raw; }
    __device__ float get(int i) const
    {
        const uint32_t w = (&raw.x)[i >> 1];
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    __device__ void set2(int i, float lo, float hi)
    {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        (&raw.x)[i >> 1] = *reinterpret_cast<uint32_t *>(&v);
    }
};
template <> struct Vec8<float> {
    float4 a, b;
    __device__ void load(const float *p) { a = *reinterpret_cast<const float4 *>(p); b = *reinterpret_cast<const float4 *>(p + 4); }
    __device__ void store(float *p) const { *reinterpret_cast<float4 *>(p) = a; *reinterpret_cast<float4 *>(p + 4) = b; }
    __device__ float get(int i) const { return i < 4 ? (&a.x)[i] : (&b.x)[i - 4]; }
    __device__ void set2(int i, float lo, float hi)
    {
        if (i < 4) { (&a.x)[i] = lo; (&a.x)[i + 1] = hi; } else { (&b.x)[i - 4] = lo; (&b.x)[i - 3] = hi; }
    }
};

template <typename T>
__global__ void __launch_bounds__(256)
merge_kernel(int64_t n_items /* rows * hq * d / 8 */, int d8, const T *o_a, const float *lse_a, const T *o_b,
             const float *lse_b, T *o, float *lse)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_items; i += stride) {
        const int64_t rh = i / d8;                              // (row, head)
        const float la = lse_a[rh], lb = lse_b[rh];
        const float m = fmaxf(la, lb);
        const float ms = m == -INFINITY ? 0.f : m;
        const float wa = __expf(la - ms), wb = __expf(lb - ms);
        const float z = wa + wb;
        const float inv = z > 0.f ? 1.f / z : 0.f;
        Vec8<T> va, vb, vo;
        va.load(o_a + i * 8);
        vb.load(o_b + i * 8);
#pragma unroll
        for (int c = 0; c < 8; c += 2)
            vo.set2(c, (va.get(c) * wa + vb.get(c) * wb) * inv, (va.get(c + 1) * wa + vb.get(c + 1) * wb) * inv);
        vo.store(o + i * 8);
        if (lse && i - rh * d8 == 0) lse[rh] = z > 0.f ? ms + logf(z) : -INFINITY;
    }
}

cudaError_t launch_merge(int dtype, int64_t n_rows, int hq, int d, const void *o_a, const float *lse_a, const void *o_b,
                         const float *lse_b, void *o, float *lse, int sm_count, cudaStream_t s, int64_t *launches)
{
    const int64_t n_items = n_rows * hq * (d / 8);
    if (n_items == 0) return cudaSuccess;
    int64_t blocks = (n_items + 255) / 256;
    if (blocks > (int64_t)sm_count * 16) blocks = (int64_t)sm_count * 16;
    if (dtype == FEDATTN_BF16)
        merge_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, s>>>(n_items, d / 8, (const __nv_bfloat16 *)o_a, lse_a,
                                                                     (const __nv_bfloat16 *)o_b, lse_b, (__nv_bfloat16 *)o, lse);
    else
        merge_kernel<float><<<(unsigned)blocks, 256, 0, s>>>(n_items, d / 8, (const float *)o_a, lse_a, (const float *)o_b, lse_b,
                                                             (float *)o, lse);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace fedattn
