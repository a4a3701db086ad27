// bf16 split-KV decode (head_dim 128): one new query token per participant over cached K/V.
// HBM-bound: each K/V row is read once.  The query rows that share a KV head -- the g = Hq/Hkv
// grouped heads of one participant (LOCAL), or of all participants (SYNC, one shared global
// cache) -- are stacked into 16-row tiles so that QK^T and PV run on the tensor cores
// (mma.sync m16n8k16), which keeps the 32 flop/byte of the sync step far below the memory time.
// K/V tiles of 64 keys stream through a 3-stage cp.async pipeline with a 16-byte-chunk XOR
// swizzle (conflict-free ldmatrix).  Row max / row sum are reduced with warp shuffles inside
// each 4-lane quad.  Each CTA handles one (cache, KV head, split) and leaves an unnormalised
// partial (m, l, o) in its shared memory.  The splits of one (cache, KV head) are launched as
// thread-block clusters of up to 8 CTAs, which merge their partials through distributed shared
// memory (each CTA of the cluster takes a share of the rows).  If a (cache, KV head) spans several
// clusters, the cluster results go to global scratch and the CTA that arrives last for its rows
// merges them, so a decode step is one launch and no CTA ever spins on another.
#include <cooperative_groups.h>
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
constexpr int kMaxCluster = 8;                          // CTAs per cluster (portable maximum)
constexpr int kMaxSlots = 16;                           // clusters per (cache, KV head): partials in global scratch
constexpr int kCtaPartOffset = 72 * 1024;               // byte offset of the CTA's merged partial in shared memory

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


// Merges the n cluster results (slots 0 .. n-1, n <= kMaxSlots) of `rows` stacked query rows row0,
// row0 + row_step, ... of one (cache, KV head), normalises and writes o / lse.  Called by every thread
// of the CTA.  Each thread owns 4 output columns of a row and reads every slot's (m, l) itself, so all
// loads are issued at once and there is no barrier.
template <int kThreads>
__device__ __forceinline__ void merge_slots(const DecodeParams &p, int n, int cache, int kvh, int row0, int row_step,
                                            int rows)
{
    const int g = p.hq / p.hkv;
    for (int i = threadIdx.x; i < rows * (kD / 4); i += kThreads) {
        const int rr = i / (kD / 4), c4 = i - rr * (kD / 4);
        const int srow = row0 + rr * row_step;
        const int part = p.sync ? srow / g : cache;
        const int head = kvh * g + (p.sync ? srow % g : srow);
        const size_t orow = (size_t)part * p.hq + head;
        const float *src = p.partial + orow * n * kPartialStride;
        float mm = -INFINITY, ll = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k0 = 0; k0 < n; k0 += 4) {
            float2 ml[4];
            float4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k0 + k < n) {
                    ml[k] = __ldcg(reinterpret_cast<const float2 *>(src + (size_t)(k0 + k) * kPartialStride));
                    v[k] = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)(k0 + k) * kPartialStride + 4 + c4 * 4));
                }
            float mn = mm;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k0 + k < n) mn = fmaxf(mn, ml[k].x);
            const float ms = mn == -INFINITY ? 0.f : mn;
            const float f0 = ex2(mm - ms);                      // 0 on the first chunk (mm = -inf)
            ll *= f0; a.x *= f0; a.y *= f0; a.z *= f0; a.w *= f0;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k0 + k < n) {
                    const float f = ex2(ml[k].x - ms);
                    ll += ml[k].y * f;
                    a.x += v[k].x * f; a.y += v[k].y * f; a.z += v[k].z * f; a.w += v[k].w * f;
                }
            mm = mn;
        }
        const float inv = ll > 0.f ? 1.f / ll : 0.f;
        __nv_bfloat162 lo = __floats2bfloat162_rn(a.x * inv, a.y * inv), hi = __floats2bfloat162_rn(a.z * inv, a.w * inv);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t *>(&lo); w.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.o) + orow * kD + c4 * 4) = w;
        if (c4 == 0 && p.lse) p.lse[orow] = ll > 0.f ? (mm + log2f(ll)) * 0.6931471805599453f : -INFINITY;
    }
}

// true in exactly one CTA: the last of `expected` to call this for the counter (which it resets to zero)
__device__ __forceinline__ bool arrive_last(int32_t *ctr, int expected, int *s_flag)
{
    __threadfence();                                            // this CTA's partials before its arrival
    __syncthreads();
    if (threadIdx.x == 0) {
        const int prev = atomicAdd(ctr, 1);
        *s_flag = prev == expected - 1;
        if (*s_flag) *ctr = 0;                                  // ready for the next call
    }
    __syncthreads();
    const bool last = *s_flag != 0;
    if (last) __threadfence();                                  // the others' partials after their arrivals
    return last;
}

#ifdef FEDATTN_DTRACE
// Debug build only: cycle stamps of the phases of every CTA's thread 0, [cta][event].
__device__ long long g_dtrace[1024 * 8];
#define DTRACE(e) do { if (threadIdx.x == 0) { const int b_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); if (b_ < 1024) g_dtrace[b_ * 8 + (e)] = clock64(); } } while (0)
#else
#define DTRACE(e) do { } while (0)
#endif

// grid: x = split, y = KV head, z = cache * n_chunks + chunk   (cache = participant for LOCAL, 0 for SYNC)
// block: 128 threads = 4 warps over (key slice, M-tile).  kMTiles == 1: 4 key slices of 16 keys of
// every 64-key tile.  kMTiles == 2: 2 key slices of 32 keys x the 2 M-tiles, one M-tile per warp, so
// the slice merge at the end moves half as much (K/V fragments are read by two warps instead).
template <int kMTiles>
__global__ void __launch_bounds__(128, 2)
decode_split_kernel(const DecodeParams p, int n_splits, int n_chunks)
{
    constexpr int kSlices = 4 / kMTiles;                        // key slices per tile
    constexpr int kSteps = 4 / kSlices;                         // 16-key steps per warp and tile
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slice = warp % kSlices, mt = warp / kSlices;     // this warp's key slice and M-tile
    DTRACE(0);
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
    __syncthreads();
    DTRACE(3);

    // ---- merge the key slices (warps) into this CTA's partial, kept in shared memory ----
    // 1. every warp posts the exponent references of its rows; 2. every thread rescales its own
    // accumulators to the common reference of its rows (in registers) and posts them; 3. the slices
    // are summed with 16-byte reads.
    float *red = reinterpret_cast<float *>(smem);               // [slice][16 kMTiles rows][kPartialStride]
    float *sm_m = reinterpret_cast<float *>(smem + 68 * 1024);  // [slice][16 kMTiles rows]
    float *sm_l = sm_m + 4 * 16 * kMTiles;
    float *cta_part = reinterpret_cast<float *>(smem + kCtaPartOffset);   // [16 kMTiles rows][kPartialStride]
    constexpr int kRows = 16 * kMTiles;
    // only the rows that carry a query take part (LOCAL mode stacks g rows into a 16-row tile)
    const int rows_here = min(kRows, rows_total - chunk * kRows);
    const int ra = mt * 16 + (lane >> 2), rb = ra + 8;          // this thread's rows inside the CTA
    if ((lane & 3) == 0) {
        sm_m[slice * kRows + ra] = m0;
        sm_m[slice * kRows + rb] = m1;
    }
    __syncthreads();
    {
        float ma = -INFINITY, mb = -INFINITY;
#pragma unroll
        for (int sl = 0; sl < kSlices; ++sl) { ma = fmaxf(ma, sm_m[sl * kRows + ra]); mb = fmaxf(mb, sm_m[sl * kRows + rb]); }
        const float fa = ex2(m0 - (ma == -INFINITY ? 0.f : ma)), fb = ex2(m1 - (mb == -INFINITY ? 0.f : mb));
        // quad-reduce l (each lane of a quad summed different keys)
        float la = l0, lb = l1;
        la += __shfl_xor_sync(0xffffffffu, la, 1); la += __shfl_xor_sync(0xffffffffu, la, 2);
        lb += __shfl_xor_sync(0xffffffffu, lb, 1); lb += __shfl_xor_sync(0xffffffffu, lb, 2);
        if ((lane & 3) == 0) { sm_l[slice * kRows + ra] = la * fa; sm_l[slice * kRows + rb] = lb * fb; }
        float *w0 = red + ((size_t)slice * kRows + ra) * kPartialStride + 4 + (lane & 3) * 2;
        float *w1 = w0 + 8 * kPartialStride;
        if (ra < rows_here) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *reinterpret_cast<float2 *>(w0 + i * 8) = make_float2(acc[i][0] * fa, acc[i][1] * fa);
        }
        if (rb < rows_here) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *reinterpret_cast<float2 *>(w1 + i * 8) = make_float2(acc[i][2] * fb, acc[i][3] * fb);
        }
    }
    __syncthreads();
    for (int i = tid; i < rows_here * (kD / 4); i += 128) {
        const int rr = i / (kD / 4), c4 = i - rr * (kD / 4);
        float4 a = *reinterpret_cast<const float4 *>(red + (size_t)rr * kPartialStride + 4 + c4 * 4);
#pragma unroll
        for (int sl = 1; sl < kSlices; ++sl) {
            const float4 v = *reinterpret_cast<const float4 *>(red + ((size_t)sl * kRows + rr) * kPartialStride + 4 + c4 * 4);
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        float *dst = cta_part + rr * kPartialStride;
        *reinterpret_cast<float4 *>(dst + 4 + c4 * 4) = a;
        if (c4 == 0) {
            float mm = -INFINITY, ll = 0.f;
#pragma unroll
            for (int sl = 0; sl < kSlices; ++sl) { mm = fmaxf(mm, sm_m[sl * kRows + rr]); ll += sm_l[sl * kRows + rr]; }
            dst[0] = mm; dst[1] = ll;
        }
    }

    // ---- cluster merge through distributed shared memory: rank k takes rows k, k + cs, ... ----
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int ncl = n_splits / cs, ci = split / cs;            // clusters per (cache, KV head); this cluster
    const int row0 = chunk * kMTiles * 16, rows = min(kMTiles * 16, rows_total - row0);
    const int my_rows = rows > rank ? (rows - rank + cs - 1) / cs : 0;
    auto out_row = [&](int srow) -> size_t {
        const int part = p.sync ? srow / g : cache;
        const int head = kvh * g + (p.sync ? srow % g : srow);
        return (size_t)part * p.hq + head;
    };
    DTRACE(4);
    cluster.sync();                                             // every CTA's partial is in place
    for (int i = tid; i < my_rows * (kD / 4); i += 128) {
        const int k = i / (kD / 4), c4 = i - k * (kD / 4);
        const int rr = rank + k * cs;
        float2 ml[kMaxCluster];
        float4 v[kMaxCluster];
#pragma unroll
        for (int q = 0; q < kMaxCluster; ++q)
            if (q < cs) {
                const float *peer = cluster.map_shared_rank(cta_part, q) + rr * kPartialStride;
                ml[q] = *reinterpret_cast<const float2 *>(peer);
                v[q] = *reinterpret_cast<const float4 *>(peer + 4 + c4 * 4);
            }
        float mm = -INFINITY;
#pragma unroll
        for (int q = 0; q < kMaxCluster; ++q)
            if (q < cs) mm = fmaxf(mm, ml[q].x);
        const float ms = mm == -INFINITY ? 0.f : mm;
        float ll = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < kMaxCluster; ++q)
            if (q < cs) {
                const float f = ex2(ml[q].x - ms);
                ll += ml[q].y * f;
                a.x += v[q].x * f; a.y += v[q].y * f; a.z += v[q].z * f; a.w += v[q].w * f;
            }
        const size_t orow = out_row(row0 + rr);
        if (ncl == 1) {
            const float inv = ll > 0.f ? 1.f / ll : 0.f;
            __nv_bfloat162 lo = __floats2bfloat162_rn(a.x * inv, a.y * inv), hi = __floats2bfloat162_rn(a.z * inv, a.w * inv);
            uint2 w;
            w.x = *reinterpret_cast<uint32_t *>(&lo); w.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.o) + orow * kD + c4 * 4) = w;
            if (c4 == 0 && p.lse) p.lse[orow] = ll > 0.f ? (mm + log2f(ll)) * 0.6931471805599453f : -INFINITY;
        } else {
            float *dst = p.partial + (orow * ncl + ci) * kPartialStride;
            *reinterpret_cast<float4 *>(dst + 4 + c4 * 4) = a;
            if (c4 == 0) { dst[0] = mm; dst[1] = ll; }
        }
    }
    // This CTA is done reading its peers; it may not exit before they are done reading it.  Arrive now,
    // wait at the very end: what follows does not touch distributed shared memory.
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    DTRACE(5);

    // ---- several clusters per (cache, KV head): the last to arrive for these rows merges them ----
    __shared__ int s_flag;
    if (ncl > 1 && my_rows > 0) {                               // CTA-uniform
        const int source = blockIdx.z * gridDim.y + kvh;
        const bool last = arrive_last(p.counters + source * kMaxCluster + rank, ncl, &s_flag);
        DTRACE(6);
        if (last) {
            merge_slots<128>(p, ncl, cache, kvh, row0 + rank, cs, my_rows);
            DTRACE(7);
        }
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
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

// Grid rule shared by both entry points.  Splits are chosen so that the whole grid is resident at
// once (two CTAs per SM): a grid slightly larger than that would run a nearly empty second wave.
// The splits of one (cache, KV head) form clusters of cs = 1, 2, 4 or 8 CTAs along grid.x.
static cudaError_t launch_decode_split(const DecodeParams &p_in, int sm_count, int max_slots, cudaStream_t s,
                                       int64_t *launches)
{
    DecodeParams p = p_in;
    const int g = p.hq / p.hkv;
    p.g_shift = -1;
    for (int sh = 0; sh < 16; ++sh)
        if ((1 << sh) == g) p.g_shift = sh;
    const int rows_total = p.sync ? p.n_part * g : g;
    const int m_tiles = rows_total > 16 ? 2 : 1;
    const int n_chunks = (rows_total + 16 * m_tiles - 1) / (16 * m_tiles);
    const int caches = p.sync ? 1 : p.n_part;
    const int sources = caches * p.hkv * n_chunks;
    const int tiles = (p.max_kv_len + kTileKeys - 1) / kTileKeys;
    int n_splits = 2 * sm_count / sources;                     // rounded down: one wave
    if (n_splits > tiles / 2) n_splits = tiles / 2;            // at least two tiles per split
    if (n_splits < 1) n_splits = 1;
    int cs = 1;
    while (cs * 2 <= kMaxCluster && cs * 2 <= n_splits) cs *= 2;
    int ncl = n_splits / cs;
    if (ncl > max_slots) ncl = max_slots;
    if (ncl > kMaxSlots) ncl = kMaxSlots;
    // several clusters per source meet through the arrival counters (kMaxCluster per source); with more
    // sources than counters every source keeps to one cluster, which needs none
    if (ncl > 1 && (int64_t)sources * kMaxCluster > kDecodeCounters) ncl = 1;
    n_splits = ncl * cs;
    if (ncl > 1 && (size_t)p.n_part * p.hq * ncl * kPartialStride * sizeof(float) > p.partial_bytes)
        return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(n_splits, p.hkv, caches * n_chunks);
    cfg.blockDim = dim3(128, 1, 1);
    cfg.dynamicSmemBytes = kStages * kStageBytes;              // 96 KB (also covers the merge buffers)
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = cs; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaError_t e = m_tiles == 1 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<1>, p, n_splits, n_chunks)
                                 : cudaLaunchKernelEx(&cfg, decode_split_kernel<2>, p, n_splits, n_chunks);
    if (launches) ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

static cudaError_t set_decode_smem_attr()
{
    const int smem = kStages * kStageBytes;
    cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_split_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
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
    return launch_decode_split(p, ctx->sm_count, kMaxSlots, s, launches);
}

}  // namespace fedattn

// ---- decode without any allocation ------------------------------------------------------------------
// Some callers cannot allocate device memory at all: code that runs inside a region where the
// allocator must not be entered (a latency-critical serving loop, a plugin that is handed its
// buffers and nothing else), or code that cannot create the workspace-owning context because it
// is not allowed to call cudaMalloc.  For them the split-KV partials live in a fixed array that is
// part of the library image: every GPU that loads the library holds these 2.07 MiB until exit.
namespace fedattn {
namespace {

constexpr int kStaticMaxRows = 256;     // n_participants * n_q_heads
constexpr int kStaticMaxSlots = 16;       // cluster results per (cache, KV head)
constexpr size_t kStaticScratchFloats = (size_t)kStaticMaxRows * kStaticMaxSlots * kPartialStride;

static __device__ __align__(256) float g_decode_scratch[kStaticScratchFloats];
// arrival counters of the split merge; zero at load, and every call leaves them zero again
static __device__ __align__(256) int32_t g_decode_counters[kDecodeCounters];

// Device address of g_decode_scratch per device.  In host code the array's name is only a handle
// for the runtime, so the address handed to the kernels comes from cudaGetSymbolAddress, taken
// once per device with that device current.
float *g_decode_scratch_ptr[64] = {};
int32_t *g_decode_counters_ptr[64] = {};
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
        int32_t *cptr = nullptr;
        if (cudaGetSymbolAddress((void **)&cptr, g_decode_counters) != cudaSuccess || !cptr) return FEDATTN_ERR_CUDA;
        g_decode_sm_count[dev] = sms;
        g_decode_counters_ptr[dev] = cptr;
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
    p.counters = g_decode_counters_ptr[dev];

    // same grid rule as the workspace-backed call, with the split count capped to the built-in scratch
    if (launch_decode_split(p, g_decode_sm_count[dev], kStaticMaxSlots, static_cast<cudaStream_t>(stream), nullptr) !=
        cudaSuccess)
        return FEDATTN_ERR_CUDA;
    return FEDATTN_OK;
}
