// bf16 split-KV decode (head_dim 128): one new query token per participant over cached K/V.
// HBM-bound: each K/V row is read once.  The query rows that share a KV head -- the g = Hq/Hkv
// grouped heads of one participant (LOCAL), or of all participants (SYNC, one shared global
// cache) -- are stacked into 16-row tiles so that QK^T and PV run on the tensor cores
// (mma.sync m16n8k16), which keeps the 32 flop/byte of the sync step far below the memory time.
// K/V tiles of 64 keys stream through a 3-stage cp.async pipeline with a 16-byte-chunk XOR
// swizzle (conflict-free ldmatrix).  Row max / row sum are reduced with warp shuffles inside
// each 4-lane quad.
//
// Two launches per decode call, chained by programmatic dependent launch:
//   decode_stream_kernel  one CTA per (cache, KV head, split); every warp walks its key slice of the
//                         split's tiles and leaves an unnormalised partial (m, l, o) per query row in
//                         global scratch.  Nothing is merged here, so a CTA ends with its last tile.
//   decode_merge_kernel   one CTA per output row: its partials (splits x key slices) are rescaled to a
//                         common exponent reference, summed, normalised and written.  Its CTAs are
//                         resident and waiting before the stream kernel ends, so the merge starts the
//                         moment the last partial is visible.
// Both kernels release their dependents as soon as they start.  The stream kernel reads its inputs
// (q, kv_len, K/V) right away and waits for the preceding grid of the stream (griddepcontrol.wait)
// only before its first write, the partials, which the merge of the previous call may still be
// reading.  In a run of back-to-back decode calls a stream CTA of call i+1 therefore takes the seat of
// a stream CTA of call i the moment that one ends, and the late CTAs, the flush and the merge of
// call i are hidden behind the next call's streaming.  Reading before the wait is sound because the
// only grids that release dependents early are this library's own, and they write nothing but their
// outputs and the scratch: the launcher checks the inputs of a call against the outputs of the recent
// calls of that kind and falls back to waiting first when they overlap (early_start.cu).  No CTA ever
// waits on another CTA.
#include <string.h>

#include "common.cuh"

namespace fedattn {

namespace {

constexpr int kD = 128;
constexpr int kTileKeys = 64;
constexpr int kStages = 3;
constexpr int kTileBytes = kTileKeys * kD * 2;          // 16 KB (K or V)
constexpr int kStageBytes = 2 * kTileBytes;             // K + V
constexpr int kPartialStride = kD + 4;                  // m, l, 2 pad, o[128]: o is 16-byte aligned
constexpr float kRescaleThreshold = 8.0f;               // log2 units
constexpr int kMaxSlots = 64;                           // partials per output row: splits x key slices of a CTA
constexpr int kMergeGroups = 4;                         // the merge kernel sums a row's partials in this many groups

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int sz = valid ? 16 : 0;      // src-size 0 => zero fill
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// byte offset of 16-byte chunk `chunk` (0..15) of key row `row` inside a swizzled [64][128] bf16 tile
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

}  // namespace


#ifdef FEDATTN_DTRACE
// Debug build only: cycle stamps of the phases of every CTA's thread 0, [cta][event].
__device__ long long g_dtrace[1024 * 8];
#define DTRACE(e) do { if (threadIdx.x == 0) { const int b_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); if (b_ < 1024) g_dtrace[b_ * 8 + (e)] = clock64(); } } while (0)
#else
#define DTRACE(e) do { } while (0)
#endif

// grid: x = split, y = KV head, z = cache * n_chunks + chunk   (cache = participant for LOCAL, 0 for SYNC)
// block: 128 threads = 4 warps over (key slice, M-tile).  kMTiles == 1: 4 key slices of 16 keys of
// every 64-key tile.  kMTiles == 2: 2 key slices of 32 keys x the 2 M-tiles, one M-tile per warp (K/V
// fragments are read by two warps), which halves the partials per output row.
// Partial of output row r, slot s = split * kSlices + slice:  partial[(r * n_slots + s) * kPartialStride]
// = { m (log2 domain, scale included), l, -, -, o[128] }, unnormalised.
template <int kMTiles>
__global__ void __launch_bounds__(128, 2)
decode_stream_kernel(const DecodeParams p, int n_splits, int n_chunks)
{
    constexpr int kSlices = 4 / kMTiles;                        // key slices per tile
    constexpr int kSteps = 4 / kSlices;                         // 16-key steps per warp and tile
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slice = warp % kSlices, mt = warp / kSlices;     // this warp's key slice and M-tile
    DTRACE(0);
    // The inputs are read before the preceding grid of the stream is known to be complete unless the
    // launcher found that they may be its outputs.  The merge kernel of this call may take its seats.
    if (!p.early) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int split = blockIdx.x, kvh = blockIdx.y;
    const int cache = blockIdx.z / n_chunks, chunk = blockIdx.z - cache * n_chunks;
    const int g = p.hq / p.hkv;
    const int rows_total = p.sync ? p.n_part * g : g;          // query rows sharing this cache + KV head

    const int len = p.sync ? p.kv_len[0] : p.kv_len[cache];
    const int tiles_total = (len + kTileKeys - 1) / kTileKeys;
    const int tiles_per_split = (tiles_total + n_splits - 1) / n_splits;
    const int tile_lo = min(split * tiles_per_split, tiles_total);
    const int tile_hi = min(tile_lo + tiles_per_split, tiles_total);
    const int n_tiles = tile_hi - tile_lo;

    const size_t tok_stride = (size_t)p.hkv * kD;              // elements
    const __nv_bfloat16 *Kb = reinterpret_cast<const __nv_bfloat16 *>(p.k) +
                              (p.sync ? 0 : (size_t)cache * p.cache_stride) + (size_t)kvh * kD;
    const __nv_bfloat16 *Vb = reinterpret_cast<const __nv_bfloat16 *>(p.v) +
                              (p.sync ? 0 : (size_t)cache * p.cache_stride) + (size_t)kvh * kD;

    // stacked row -> (participant, query head)
    auto q_ptr = [&](int srow) -> const __nv_bfloat16 * {
        if (srow >= rows_total) return nullptr;
        int part = cache, sub = srow;
        if (p.sync) {                                           // srow = part * g + sub
            if (p.g_shift >= 0) { part = srow >> p.g_shift; sub = srow & (g - 1); }
            else { part = srow / g; sub = srow - part * g; }
        }
        const int head = kvh * g + sub;
        return reinterpret_cast<const __nv_bfloat16 *>(p.q) + ((size_t)part * p.hq + head) * kD;
    };

    // K and V tiles: 64 rows x 16 chunks of 16 bytes each.  Thread tid copies chunk (tid & 15) of rows
    // (tid >> 4) + 8 i, i = 0..7; the row's swizzle term (row & 7) is the same for all i, so the global
    // and shared offsets are fixed per thread up to a multiple of 8 rows.  Rows past `len` are zero-filled.
    const int ld_row = tid >> 4, ld_ch = tid & 15;
    const __nv_bfloat16 *ld_k = Kb + (size_t)ld_row * tok_stride + ld_ch * 8, *ld_v = Vb + (size_t)ld_row * tok_stride + ld_ch * 8;
    const uint32_t ld_s = smem_u32(smem) + swz(ld_row, ld_ch);
    auto load_tile = [&](int t, int stage) {
        const int key0 = (tile_lo + t) * kTileKeys;
        const uint32_t sK = ld_s + stage * kStageBytes, sV = sK + kTileBytes;
        const size_t base = (size_t)key0 * tok_stride;
        const int n_ok = len - key0 - ld_row;                  // rows ld_row + 8 i with 8 i < n_ok exist
#pragma unroll
        for (int i = 0; i < kTileKeys / 8; ++i) {
            const bool ok = 8 * i < n_ok;
            const size_t off = ok ? base + (size_t)(8 * i) * tok_stride : 0;
            cp_async16(sK + i * 8 * 256, ld_k + off, ok);
            cp_async16(sV + i * 8 * 256, ld_v + off, ok);
        }
    };

    const float sl2 = p.scale * 1.4426950408889634f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows lane/4 and lane/4 + 8 of this warp's M-tile
    float acc[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

    // Q rows of this chunk -> shared memory (in the third stage's buffer, which the first tile loads do
    // not touch), same swizzle as the K/V tiles; rows past rows_total are zero
    {
        const uint32_t sQ = smem_u32(smem) + (kStages - 1) * kStageBytes;
#pragma unroll
        for (int i = tid; i < 16 * kMTiles * 16; i += 128) {
            const int row = i >> 4, ch = i & 15;
            const __nv_bfloat16 *src = q_ptr(chunk * kMTiles * 16 + row);
            cp_async16(sQ + swz(row, ch), src ? src + ch * 8 : reinterpret_cast<const __nv_bfloat16 *>(p.q), src != nullptr);
        }
        cp_async_commit();
    }
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) {
        if (s < n_tiles) load_tile(s, s);
        cp_async_commit();
    }
    // Q fragments of this warp's M-tile (A operand, 16 x 128): 8 k-steps x 4 registers
    uint32_t qf[8][4];
    cp_async_wait<kStages - 1>();                               // the Q group; the tile groups may still be in flight
    __syncthreads();
    {
        const uint32_t sQ = smem_u32(smem) + (kStages - 1) * kStageBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            // matrices: (rows 0-7, d 0-7) (rows 8-15, d 0-7) (rows 0-7, d 8-15) (rows 8-15, d 8-15)
            const int row = mt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
            const int ch = ks * 2 + (lane >> 4);
            ldmatrix_x4(qf[ks], sQ + swz(row, ch));
        }
    }
    DTRACE(1);
    for (int t = 0; t < n_tiles; ++t) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        if (t == 0) DTRACE(2);
        if (t + kStages - 1 < n_tiles) load_tile(t + kStages - 1, (t + kStages - 1) % kStages);
        cp_async_commit();

        const uint32_t sK = smem_u32(smem) + (t % kStages) * kStageBytes, sV = sK + kTileBytes;
#pragma unroll
        for (int step = 0; step < kSteps; ++step) {
            const int krow0 = (slice * kSteps + step) * 16;
            // ---- S = Q K^T for 16 keys: two n-tiles of 8 keys ----
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                // matrices: (keys 0-7, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 0-7) (keys 8-15, d 8-15)
                const int row = krow0 + (lane & 7) + ((lane >> 4) << 3);
                const int ch = ks * 2 + ((lane >> 3) & 1);
                uint32_t b[4];
                ldmatrix_x4(b, sK + swz(row, ch));
                mma_bf16(s0, qf[ks], b[0], b[1]);
                mma_bf16(s1, qf[ks], b[2], b[3]);
            }
            // ---- mask keys past the end, online softmax (rows lane/4 and lane/4+8) ----
            const int key = (tile_lo + t) * kTileKeys + krow0 + (lane & 3) * 2;
            const bool ok[4] = {key < len, key + 1 < len, key + 8 < len, key + 9 < len};
            float v[8] = {s0[0], s0[1], s1[0], s1[1], s0[2], s0[3], s1[2], s1[3]};   // row0: v[0..3], row1: v[4..7]
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                v[i] = ok[i] ? v[i] * sl2 : -INFINITY;
                v[i + 4] = ok[i] ? v[i + 4] * sl2 : -INFINITY;
            }
            float mx0 = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3])), mx1 = fmaxf(fmaxf(v[4], v[5]), fmaxf(v[6], v[7]));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            // The exponent reference of a row moves only when its maximum grew by more than 2^8 (or is
            // still unset); the accumulators are rescaled only then.  The final normalisation uses the
            // same reference, so the result is exact up to rounding.
            const bool g0 = mx0 > m0 + kRescaleThreshold, g1 = mx1 > m1 + kRescaleThreshold;
            if (__any_sync(0xffffffffu, g0 || g1)) {
                const float mn0 = g0 ? mx0 : m0, mn1 = g1 ? mx1 : m1;
                const float a0 = g0 ? ex2(m0 - mn0) : 1.f, a1 = g1 ? ex2(m1 - mn1) : 1.f;
                m0 = mn0; m1 = mn1;
                l0 *= a0; l1 *= a1;
#pragma unroll
                for (int i = 0; i < 16; ++i) { acc[i][0] *= a0; acc[i][1] *= a0; acc[i][2] *= a1; acc[i][3] *= a1; }
            }
            const float ms0 = m0 == -INFINITY ? 0.f : m0, ms1 = m1 == -INFINITY ? 0.f : m1;
            float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                v[i] = ex2(v[i] - ms0); ps0 += v[i];
                v[i + 4] = ex2(v[i + 4] - ms1); ps1 += v[i + 4];
            }
            l0 += ps0; l1 += ps1;
            // P as A operand (16 rows x 16 keys)
            const uint32_t pf[4] = {pack_bf16(v[0], v[1]), pack_bf16(v[4], v[5]), pack_bf16(v[2], v[3]), pack_bf16(v[6], v[7])};
            // ---- O += P V ----
#pragma unroll
            for (int nd = 0; nd < 8; ++nd) {
                // matrices: (keys 0-7, d 0-7) (keys 8-15, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 8-15) of d block nd*16
                const int row = krow0 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int ch = nd * 2 + (lane >> 4);
                uint32_t b[4];
                ldmatrix_x4_trans(b, sV + swz(row, ch));
                mma_bf16(acc[2 * nd], pf, b[0], b[1]);
                mma_bf16(acc[2 * nd + 1], pf, b[2], b[3]);
            }
        }
    }
    cp_async_wait<0>();
    DTRACE(3);


    // the scratch may still be read by the merge of the previous call: the preceding grid must be complete
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ---- every warp leaves the partial of its key slice: nothing is merged here ----
    constexpr int kRows = 16 * kMTiles;
    const int rows_here = min(kRows, rows_total - chunk * kRows);   // LOCAL stacks g rows into a 16-row tile
    const int n_slots = n_splits * kSlices, slot = split * kSlices + slice;
    auto out_row = [&](int srow) -> size_t {
        int part = cache, sub = srow;
        if (p.sync) {
            if (p.g_shift >= 0) { part = srow >> p.g_shift; sub = srow & (g - 1); }
            else { part = srow / g; sub = srow - part * g; }
        }
        return (size_t)part * p.hq + kvh * g + sub;
    };
    // each lane of a quad summed different keys
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const int ra = mt * 16 + (lane >> 2), rb = ra + 8;          // this thread's rows inside the CTA
    if (ra < rows_here) {
        float *dst = p.partial + (out_row(chunk * kRows + ra) * n_slots + slot) * kPartialStride;
        if ((lane & 3) == 0) *reinterpret_cast<float2 *>(dst) = make_float2(m0, l0);
        dst += 4 + (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < 16; ++i) *reinterpret_cast<float2 *>(dst + i * 8) = make_float2(acc[i][0], acc[i][1]);
    }
    if (rb < rows_here) {
        float *dst = p.partial + (out_row(chunk * kRows + rb) * n_slots + slot) * kPartialStride;
        if ((lane & 3) == 0) *reinterpret_cast<float2 *>(dst) = make_float2(m1, l1);
        dst += 4 + (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < 16; ++i) *reinterpret_cast<float2 *>(dst + i * 8) = make_float2(acc[i][2], acc[i][3]);
    }
    DTRACE(4);
}

// A CTA takes output rows (participant, query head) blockIdx.x, blockIdx.x + gridDim.x, ...: thread =
// (group of slots, 4 output columns).  Every thread folds its group's partials, four loads in flight at
// a time; the groups meet in shared memory.  The grid is at most one CTA per SM and a CTA is small (128
// threads, few registers, 2 KB of shared memory), so the whole grid is resident beside the stream CTAs
// at once: the next call's stream kernel can only be launched when every CTA of this grid has started.
__global__ void __launch_bounds__(kMergeGroups * (kD / 4), 7)
decode_merge_kernel(const DecodeParams p, int n_slots, int n_rows)
{
    __shared__ float4 s_acc[kMergeGroups][kD / 4];
    __shared__ float2 s_ml[kMergeGroups];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");         // the partials of this call
    const int c4 = threadIdx.x & (kD / 4 - 1), grp = threadIdx.x / (kD / 4);
    for (size_t orow = blockIdx.x; orow < (size_t)n_rows; orow += gridDim.x) {
    const int per = (n_slots + kMergeGroups - 1) / kMergeGroups;
    const int s0 = grp * per, s1 = min(s0 + per, n_slots);
    const float *src = p.partial + orow * n_slots * kPartialStride;
    float mm = -INFINITY, ll = 0.f;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = s0; k0 < s1; k0 += 4) {
        float2 ml[4];
        float4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (k0 + k < s1) {
                ml[k] = __ldcg(reinterpret_cast<const float2 *>(src + (size_t)(k0 + k) * kPartialStride));
                v[k] = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)(k0 + k) * kPartialStride + 4 + c4 * 4));
            }
        float mn = mm;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (k0 + k < s1) mn = fmaxf(mn, ml[k].x);
        const float ms = mn == -INFINITY ? 0.f : mn;
        const float f0 = ex2(mm - ms);                          // 0 on the first batch (mm = -inf)
        ll *= f0; a.x *= f0; a.y *= f0; a.z *= f0; a.w *= f0;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (k0 + k < s1) {
                const float f = ex2(ml[k].x - ms);              // 0 for an empty partial (m = -inf)
                ll += ml[k].y * f;
                a.x += v[k].x * f; a.y += v[k].y * f; a.z += v[k].z * f; a.w += v[k].w * f;
            }
        mm = mn;
    }
    s_acc[grp][c4] = a;
    if (c4 == 0) s_ml[grp] = make_float2(mm, ll);
    __syncthreads();
    if (grp == 0) {
        float m_all = -INFINITY;
#pragma unroll
        for (int q = 0; q < kMergeGroups; ++q) m_all = fmaxf(m_all, s_ml[q].x);
        const float mr = m_all == -INFINITY ? 0.f : m_all;
        float l_all = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < kMergeGroups; ++q) {
            const float f = ex2(s_ml[q].x - mr);
            const float4 t = s_acc[q][c4];
            l_all += s_ml[q].y * f;
            o.x += t.x * f; o.y += t.y * f; o.z += t.z * f; o.w += t.w * f;
        }
        const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
        __nv_bfloat162 lo = __floats2bfloat162_rn(o.x * inv, o.y * inv), hi = __floats2bfloat162_rn(o.z * inv, o.w * inv);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t *>(&lo); w.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.o) + orow * kD + c4 * 4) = w;
        if (c4 == 0 && p.lse) p.lse[orow] = l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
    }
    __syncthreads();                                            // the group buffers are reused by the next row
    }
}

#ifdef FEDATTN_DTRACE
extern "C" int fedattn_debug_read_dtrace(long long *host, int n)
{
    return (int)cudaMemcpyFromSymbol(host, g_dtrace, sizeof(long long) * n);
}
#endif

size_t decode_scratch_bytes(int n_part, int hq, int d, int /*sm_count*/)
{
    if (d != kD) return 0;
    return (size_t)n_part * hq * kMaxSlots * kPartialStride * sizeof(float);
}

// Grid rule shared by both entry points.  Splits are chosen so that the whole stream grid is resident
// at once (two CTAs per SM): a grid slightly larger than that would run a nearly empty second wave.
static cudaError_t launch_decode_split(const DecodeParams &p_in, int device, int sm_count, cudaStream_t s,
                                       int64_t *launches)
{
    DecodeParams p = p_in;
    {
        // may the stream kernel read its inputs before the preceding grid of the stream is complete?
        const size_t row_bytes = (size_t)p.hkv * kD * 2, qo_bytes = (size_t)p.n_part * p.hq * kD * 2;
        const size_t cache_bytes = p.sync ? (size_t)p.max_kv_len * row_bytes
                                          : ((size_t)(p.n_part - 1) * p.cache_stride * 2 + (size_t)p.max_kv_len * row_bytes);
        const MemRange in[4] = {{p.q, qo_bytes}, {p.k, cache_bytes}, {p.v, cache_bytes},
                                {p.kv_len, (p.sync ? 1 : p.n_part) * sizeof(int32_t)}};
        const MemRange out[2] = {{p.o, qo_bytes}, {p.lse, p.lse ? (size_t)p.n_part * p.hq * sizeof(float) : 0}};
        p.early = early_start(device, s, in, 4, out, 2).early ? 1 : 0;
    }
    const int g = p.hq / p.hkv;
    p.g_shift = -1;
    for (int sh = 0; sh < 16; ++sh)
        if ((1 << sh) == g) p.g_shift = sh;
    const int rows_total = p.sync ? p.n_part * g : g;
    const int m_tiles = rows_total > 16 ? 2 : 1;
    const int slices = 4 / m_tiles;                             // key slices (warps per M-tile) of a CTA
    const int n_chunks = (rows_total + 16 * m_tiles - 1) / (16 * m_tiles);
    const int caches = p.sync ? 1 : p.n_part;
    const int sources = caches * p.hkv * n_chunks;
    const int tiles = (p.max_kv_len + kTileKeys - 1) / kTileKeys;
    int n_splits = 2 * sm_count / sources;                     // rounded down: one wave
    if (n_splits > tiles / 2) n_splits = tiles / 2;            // at least two tiles per split
    if (n_splits > kMaxSlots / slices) n_splits = kMaxSlots / slices;
    if (n_splits < 1) n_splits = 1;
    const int n_slots = n_splits * slices;
    if ((size_t)p.n_part * p.hq * n_slots * kPartialStride * sizeof(float) > p.partial_bytes) return cudaErrorInvalidValue;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(n_splits, p.hkv, caches * n_chunks);
    cfg.blockDim = dim3(128, 1, 1);
    cfg.dynamicSmemBytes = kStages * kStageBytes;              // 96 KB
    cfg.stream = s;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaError_t e = m_tiles == 1 ? cudaLaunchKernelEx(&cfg, decode_stream_kernel<1>, p, n_splits, n_chunks)
                                 : cudaLaunchKernelEx(&cfg, decode_stream_kernel<2>, p, n_splits, n_chunks);
    if (launches) ++*launches;
    if (e != cudaSuccess) return e;
    const int n_rows = p.n_part * p.hq, rows_per_cta = (n_rows + sm_count - 1) / sm_count;
    cfg.gridDim = dim3((n_rows + rows_per_cta - 1) / rows_per_cta, 1, 1);
    cfg.blockDim = dim3(kMergeGroups * (kD / 4), 1, 1);
    cfg.dynamicSmemBytes = 0;
    e = cudaLaunchKernelEx(&cfg, decode_merge_kernel, p, n_slots, n_rows);
    if (launches) ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

static cudaError_t set_decode_smem_attr()
{
    const int smem = kStages * kStageBytes;
    cudaError_t e = cudaFuncSetAttribute(decode_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_stream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return e;
}

cudaError_t launch_decode_bf16(const Context *ctx, const DecodeParams &p, cudaStream_t s, int64_t *launches)
{
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        cudaError_t e = set_decode_smem_attr();
        if (e != cudaSuccess) return e;
        attr_set[ctx->device & 63] = true;
    }
    return launch_decode_split(p, ctx->device, ctx->sm_count, s, launches);
}

}  // namespace fedattn

// ---- decode without any allocation ------------------------------------------------------------------
// Some callers cannot allocate device memory at all: code that runs inside a region where the
// allocator must not be entered (a latency-critical serving loop, a plugin that is handed its
// buffers and nothing else), or code that cannot create the workspace-owning context because it
// is not allowed to call cudaMalloc.  For them the split-KV partials live in a fixed array that is
// part of the library image: every GPU that loads the library holds these 8.25 MiB until exit.
namespace fedattn {
namespace {

constexpr int kStaticMaxRows = 256;     // n_participants * n_q_heads
constexpr size_t kStaticScratchFloats = (size_t)kStaticMaxRows * kMaxSlots * kPartialStride;

static __device__ __align__(256) float g_decode_scratch[kStaticScratchFloats];

// Device address of g_decode_scratch per device.  In host code the array's name is only a handle
// for the runtime, so the address handed to the kernels comes from cudaGetSymbolAddress, taken
// once per device with that device current.
float *g_decode_scratch_ptr[64] = {};
int g_decode_sm_count[64] = {};

}  // namespace
}  // namespace fedattn

extern "C" fedattn_status fedattn_decode_noalloc(const fedattn_shape *shape, int32_t mode, const void *q,
                                                 const void *k_cache, const void *v_cache,
                                                 int64_t cache_stride_participant, const int32_t *kv_len,
                                                 int32_t max_kv_len, void *o, float *lse, fedattn_stream stream)
{
    using namespace fedattn;
    if (!shape || shape->n_participants < 1 || shape->n_q_heads < 1 || shape->n_kv_heads < 1 ||
        shape->n_q_heads % shape->n_kv_heads != 0)
        return FEDATTN_ERR_INVALID_ARG;
    if (mode != FEDATTN_DECODE_LOCAL && mode != FEDATTN_DECODE_SYNC) return FEDATTN_ERR_INVALID_ARG;
    if (!q || !o || !kv_len || max_kv_len < 0 || cache_stride_participant < 0) return FEDATTN_ERR_INVALID_ARG;
    if (max_kv_len > 0 && (!k_cache || !v_cache)) return FEDATTN_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)o | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15) return FEDATTN_ERR_INVALID_ARG;
    if (mode == FEDATTN_DECODE_LOCAL && (cache_stride_participant * 2) % 16 != 0) return FEDATTN_ERR_INVALID_ARG;
    if (shape->dtype != FEDATTN_BF16 || shape->head_dim != kD) return FEDATTN_ERR_UNSUPPORTED;
    if ((int64_t)shape->n_participants * shape->n_q_heads > kStaticMaxRows)
        return FEDATTN_ERR_WORKSPACE;          // more output rows than the built-in scratch covers
    if (!(shape->scale >= 0.f)) return FEDATTN_ERR_INVALID_ARG;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FEDATTN_ERR_CUDA;
    if (!g_decode_scratch_ptr[dev]) {
        // first call on this device: resolve the array's device address and the SM count
        float *ptr = nullptr;
        if (cudaGetSymbolAddress((void **)&ptr, g_decode_scratch) != cudaSuccess || !ptr) return FEDATTN_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            return FEDATTN_ERR_CUDA;
        if (set_decode_smem_attr() != cudaSuccess) return FEDATTN_ERR_CUDA;
        g_decode_sm_count[dev] = sms;
        g_decode_scratch_ptr[dev] = ptr;
    }

    DecodeParams p;
    memset(&p, 0, sizeof(p));
    p.q = q; p.k = k_cache; p.v = v_cache; p.o = o; p.lse = lse;
    p.n_part = shape->n_participants; p.hq = shape->n_q_heads; p.hkv = shape->n_kv_heads; p.d = kD;
    p.scale = shape->scale > 0.f ? shape->scale : 0.08838834764831845f;   // 1/sqrt(128)
    p.sync = mode == FEDATTN_DECODE_SYNC;
    p.cache_stride = cache_stride_participant; p.kv_len = kv_len; p.max_kv_len = max_kv_len;
    p.partial = g_decode_scratch_ptr[dev];
    p.partial_bytes = kStaticScratchFloats * sizeof(float);

    // same kernels and grid rule as the workspace-backed call
    if (launch_decode_split(p, dev, g_decode_sm_count[dev], static_cast<cudaStream_t>(stream), nullptr) != cudaSuccess)
        return FEDATTN_ERR_CUDA;
    return FEDATTN_OK;
}
