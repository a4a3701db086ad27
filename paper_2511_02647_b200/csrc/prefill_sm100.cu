// bf16 prefill attention for sm_100a: TMA-fed, tcgen05 tensor cores, accumulators in TMEM,
// online softmax in fp32.  Serves fedattn_local (per-participant causal attention over packed
// segments) and fedattn_sync (queries over the aggregated KV, causal on global positions).
//
// Persistent kernel, one CTA per SM.  A work item is one 128-row query tile of a PAIR of query heads
// that share a KV head (two "sub-tiles"); the CTA walks the key/value tiles the rows may see, and
// tiles that the segment descriptors or the causal mask rule out are never loaded.  Items are sorted
// by cost and dealt to the CTAs in snake order.
//
// Per KV tile j and sub-tile t:
//     S_t = Q_t K_j^T          (tcgen05.mma, A/B from shared memory, D in TMEM)
//     P_t = exp2(S_t*c - m)    (softmax threads, TMEM -> registers -> TMEM, P aliases S)
//     O_t += P_t V_j           (tcgen05.mma, A = P from TMEM, B = V from shared memory)
// The tensor pipe alternates between the sub-tiles (PV_0 S_0 | PV_1 S_1 | ...); each sub-tile has a
// softmax warpgroup of its own, so while one warpgroup is in the serial part of its visit the other
// computes and the tensor pipe works for whichever sub-tile is ready.  O stays in TMEM for the whole
// tile walk and is rescaled only when a row's running maximum grows by more than 2^8 (the final
// normalisation uses the same reference, so the result is exact up to rounding).
//
// Warp roles: warps 0-3 softmax/epilogue of sub-tile 0, warps 4-7 of sub-tile 1: thread = query row =
// TMEM lane, all 128 key columns of the S tile (read from TMEM once, held in registers for the row
// maximum and then the exponentials) and the whole row of O; nothing is exchanged between threads.  Warp 8
// TMA producer (+ TMEM allocation), warp 9 MMA issuer (the whole warp walks the loop, one elected lane
// issues); warp 10 checks the order of the key positions, warp 11 only fills that warpgroup, which
// hands most of its registers to the softmax warpgroups (setmaxnreg works on whole warpgroups).
// 2/8 of the exponentials of unmasked tiles are evaluated by a polynomial on the FMA pipe, because for
// this tile shape the ex2 unit alone is as slow as the tensor pipe.  The producer decodes every work
// item once and publishes it through shared memory for the softmax warps; finished rows leave through
// shared-memory staging and TMA stores (a warp with rows beyond its segment stores them directly).
// Every wait is bounded; on expiry the CTA sets the status word, stops waiting and runs to its normal
// end (TMEM is always released).
#include <cuda.h>

#include <stdio.h>
#include <stdlib.h>
#include <type_traits>

#include "common.cuh"

namespace fedattn {

namespace {

constexpr int kTileM = 128;          // query rows per CTA
constexpr int kTileN = 128;          // keys per KV tile
constexpr int kD = 128;              // head dim
// two softmax warpgroups, one per sub-tile.  (Both on the same S tile, split by columns with the row
// maxima exchanged through shared memory, was 2-4 % slower on dense sync; four warpgroups of 32 columns
// 20 %.)  P is handed to the MMA warp in kSplit halves of kCols keys, so that PV starts on the first.
constexpr int kSplit = 2;
constexpr int kCols = kTileN / kSplit;
constexpr int kSoftmaxThreads = 128 * kSplit;
constexpr int kThreads = kSoftmaxThreads + 128;  // then a warpgroup holding the TMA producer warp and the MMA issuer warp
// Registers move from that warpgroup to the softmax warpgroups once the roles split (setmaxnreg):
// 384 threads start with 168 each, and that allocation (3 x 168 = 504 registers per lane slot of a
// scheduler) is the pool the increases draw from.  setmaxnreg.inc waits, without limit, until the pool
// can give what it asks for, so the split must fit into it: 2 x kSoftmaxRegs + kOtherRegs <= 504; it
// keeps 8 spare.  (A 200 / 112 split asks for 512 per lane slot and never came back from the increase.)
constexpr int kSoftmaxRegs = 216, kOtherRegs = 64;
static_assert(2 * kSoftmaxRegs + kOtherRegs <= 496 && kSoftmaxRegs % 8 == 0 && kOtherRegs % 8 == 0, "register budget");
constexpr int kProducerWarp = 4 * kSplit, kMmaWarp = 4 * kSplit + 1;
static_assert(kSplit == 2 || kSplit == 4, "column split");
constexpr uint32_t kTileBytes = kTileM * kD * 2;      // 32 KB: one Q, K or V tile
constexpr uint32_t kHalfBytes = kTileBytes / 2;       // one 64-column TMA box
constexpr uint32_t kStageBytes = 32 * 128;            // output staging per softmax warp: 32 rows x 64 columns
constexpr uint32_t kSmemBytes = 6 * kTileBytes + 1024 /*alignment slack*/ + 1024 /*barriers, published items*/ +
                                2 * kSplit * 2 * kStageBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;   // S (and P, aliased) of sub-tile t at kColS + 128 t; O at kColO + 128 t
// P (bf16 pairs) of keys kCols q .. kCols q + kCols - 1 sits at S column kCols q: every 32-key chunk of P
// lands in S columns that its thread has already read
constexpr uint32_t kWaitLimit = 1u << 20;
constexpr float kRescaleThreshold = 8.0f;

struct KernelParams {
    PrefillParams p;
    int32_t ord_seg[kMaxP];          // segments sorted by query-tile count, descending
    int32_t ord_nt[kMaxP];           // their query-tile counts
    int32_t band_rank[kMaxP + 1];    // tiles ranked above band b (levels ord_nt[b+1] < lv <= ord_nt[b])
    int32_t group;                   // query heads per KV head
    uint64_t magic_per_tile, magic_ppg, magic_small[kMaxP];   // ceil(2^40 / d) for d = per_tile, ppg, 1..kMaxP
    int32_t n_qtiles;                // total query tiles
    int32_t n_items;                 // query tiles x KV heads x head pairs
    int32_t n_kt;                    // KV tiles: ceil(total_kv / kTileN)
    int32_t *status;
    int32_t o_tma;                   // the output may leave through TMA stores (tensor map encoded)
};

// Position tables of a general-position call (ints, in this order): minimum and maximum position of
// every query tile; then per KV position array (one per KV head when head-major, else one) the
// running minimum over the tiles j, j+1, ... (suffix minimum) and the running maximum over the tiles
// 0 .. j (prefix maximum) of the tile's key positions.  Both runs are monotone in j, so "tiles that
// can hold a visible key" and "tiles whose keys are all visible" are prefixes found by bisection.
// A ragged last KV tile counts as never fully visible (maximum = INT_MAX).
struct PosTables {
    const int32_t *q_min, *q_max, *suf_min, *pre_max;
};
__device__ __host__ __forceinline__ PosTables pos_tables(const int32_t *tab, int n_qtiles, int n_arrays, int n_kt)
{
    PosTables t;
    t.q_min = tab; t.q_max = tab + n_qtiles;
    t.suf_min = tab + 2 * (size_t)n_qtiles; t.pre_max = t.suf_min + (size_t)n_arrays * n_kt;
    return t;
}

#ifdef FEDATTN_TRACE
// Debug build only: cycle stamps of one CTA's pipeline events, [tile][event].
__device__ long long g_trace[64 * 8];
#define TRACE(j, e) do { if (k == 0 && blockIdx.x == gridDim.x / 2 && (j) < 64) g_trace[(j) * 8 + (e)] = clock64(); } while (0)
#else
#define TRACE(j, e) do { } while (0)
#endif

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (after flagging the status word once) when the limit is reached or
// another thread of this CTA already gave up.
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                          uint32_t limit = kWaitLimit)
{
    if (mbar_test_wait(bar, parity)) return true;        // phase already over: skip the suspending wait
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicMax(status, (int32_t)FEDATTN_ERR_TIMEOUT);
    return false;
}

// The same wait for the roles that hold few registers (producer, MMA issuer): the polling loop lives in
// one place instead of at every call site, which keeps those roles' code short.
__device__ __noinline__ bool mbar_wait_loop(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int32_t *status)
{
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicMax(status, (int32_t)FEDATTN_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ bool mbar_wait_call(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int32_t *status)
{
    if (mbar_test_wait(bar, parity)) return true;
    return mbar_wait_loop(bar, parity, abort_flag, status);
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}

__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap *map, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// [32 rows x 64 columns] from shared memory (128-byte swizzle) to the output, one bulk group per call
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, const void *src, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"((uint64_t)map), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the issuing thread's earlier bulk stores have read their shared memory
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

#define FEDATTN_TMEM_LD32(taddr, r)                                                                          \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                   \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                   \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                  \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),       \
                   "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),   \
                   "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),             \
                   "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),             \
                   "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])              \
                 : "r"(taddr) : "memory")

#define FEDATTN_TMEM_ST32(taddr, r)                                                                          \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                             \
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"                                  \
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"                         \
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),  \
                   "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),          \
                   "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),       \
                   "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),       \
                   "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory")

#define FEDATTN_TMEM_ST16(taddr, r)                                                                          \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "                                             \
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"                                 \
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),  \
                   "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),          \
                   "r"(r[14]), "r"(r[15]) : "memory")

#define FEDATTN_TMEM_LD16(taddr, r)                                                                          \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                   \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"                           \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),       \
                   "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),   \
                   "=r"(r[14]), "=r"(r[15])                                                                  \
                 : "r"(taddr) : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

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

__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// 2^x for a packed pair on the FMA/ALU pipes (no MUFU): x = n + f with n = round(x), |f| <= 1/2;
// 2^f by a degree-3 minimax polynomial (relative error 7.5e-5, far below the bf16 rounding of P),
// 2^n by adding n to the exponent field.  The magic constant 1.5 * 2^23 makes the low mantissa
// bits of x + magic hold n.  x is clamped at -125 so that the exponent arithmetic cannot wrap:
// anything smaller contributes 2^-125 instead of an even smaller value.  Needs x <= 100.
// bit (c & 7) set: column pair c takes the polynomial instead of ex2.approx.  2 of 8 pairs: 1, 2 and 3 of 8
// are within 1 % of each other (which is best depends on the board), none costs 2-3 %, 4 and 5 of 8 cost
// 2 and 5 % (the polynomial loads the ALU pipe as much as ex2 loads its own unit).
#ifndef FEDATTN_POLY_MASK
#define FEDATTN_POLY_MASK 0x11
#endif
constexpr uint32_t kPolyMask = FEDATTN_POLY_MASK;
__device__ __forceinline__ void exp2_poly_x2(uint64_t x2, float &p0, float &p1)
{
    float x0, x1;
    unpack_f32x2(x2, x0, x1);
    x0 = fmaxf(x0, -125.f); x1 = fmaxf(x1, -125.f);
    const uint64_t xc = pack_f32x2(x0, x1);
    const uint64_t magic = pack_f32x2(12582912.f, 12582912.f), neg_magic = pack_f32x2(-12582912.f, -12582912.f);
    const uint64_t neg_one = pack_f32x2(-1.f, -1.f);
    const uint64_t t2 = add_f32x2(xc, magic);
    const uint64_t f2 = fma_f32x2(add_f32x2(t2, neg_magic), neg_one, xc);
    uint64_t q2 = pack_f32x2(0.0551716685295105f, 0.0551716685295105f);
    q2 = fma_f32x2(q2, f2, pack_f32x2(0.2426111251115799f, 0.2426111251115799f));
    q2 = fma_f32x2(q2, f2, pack_f32x2(0.6932609677314758f, 0.6932609677314758f));
    q2 = fma_f32x2(q2, f2, pack_f32x2(0.9999280571937561f, 0.9999280571937561f));
    float q0, q1, t0, t1;
    unpack_f32x2(q2, q0, q1);
    unpack_f32x2(t2, t0, t1);
    p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (Q, K): rows of 64 bf16 = 128 B; a tile is two such [128 x 64] halves.
//   MN-major operand (V as B, N = head dim): 64 head-dim elements contiguous per key row;
//   lbo = distance between the two 64-wide head-dim halves.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;            // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;            // SWIZZLE_128B
    return d;
}

// Instruction descriptor, kind::f16: D fp32, A/B bf16, M = 128, N = 128.
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;                 // A, B K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);    // B (V) MN-major

// n / d for 0 <= n < 2^28 and 1 <= d <= 4096, with magic = ceil(2^40 / d)
__device__ __forceinline__ int fast_div(int n, uint64_t magic) { return (int)(((uint64_t)(uint32_t)n * magic) >> 40); }

// number of entries of the non-decreasing array pos[0..n) that are <= x
__device__ __forceinline__ int count_le(const int32_t *pos, int n, int x)
{
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(pos + mid) <= x) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// The same count, found by a converged warp together: every step probes 32 evenly spaced entries at
// once (one round trip to memory per step instead of one per halving), so 4096 entries take 3 steps.
// Every lane returns the count.
__device__ __forceinline__ int count_le_warp(const int32_t *pos, int n, int x, int lane)
{
    int lo = 0, hi = n;                                         // the count lies in [lo, hi]
    while (hi > lo) {
        const int width = hi - lo;
        if (width <= 32) {
            const bool le = lane < width && __ldg(pos + lo + lane) <= x;
            return lo + __popc(__ballot_sync(0xffffffffu, le));  // the entries <= x are a prefix
        }
        const int stride = (width + 31) >> 5;
        const int probe = min(lo + (lane + 1) * stride - 1, hi - 1);
        const int k = __popc(__ballot_sync(0xffffffffu, __ldg(pos + probe) <= x));
        if (k == 32) return hi;                                 // even the last entry is <= x
        hi = min(lo + (k + 1) * stride - 1, hi - 1);            // entry `hi` is > x: the count is at most hi
        lo = lo + k * stride;
    }
    return lo;
}

}  // namespace

// One unit of work: a 128-row query tile x one pair of query heads that share a KV head.
struct Item {
    int kvh, head0, q_row0, n_valid, seg, kv_begin, n_tiles;
    // The walk visits KV tiles 0 .. n_a-1 and then t_b0, t_b0+1, ...  (n_a == n_tiles unless the allowed
    // keys are two ranges: bidirectional remote-only attention, keys [0, a) and [b, T)).
    int n_a, t_b0, a, b;
    bool valid1;                       // the pair's second head exists (odd group size: last pair is single)
    const int32_t *kvp;                // positions of this KV head's aggregated rows (sparse sync), or null
};
__device__ __forceinline__ int tile_of(const Item &it, int j) { return j < it.n_a ? j : it.t_b0 + (j - it.n_a); }

// allowed-prefix length c(row): keys kv_begin .. kv_begin + c - 1 are visible to query row r of the tile.
// Called by a converged warp with the same r in every lane (the searches are warp-cooperative).
template <bool kSpecial>
__device__ __forceinline__ int prefix_len(const PrefillParams &p, const Item &it, int r, int lane)
{
    const int pos = it.q_row0 + r;
    const int T = (int)p.total_kv;
    if (!p.sync) {
        const int seg_len = p.cu[it.seg + 1] - p.cu[it.seg];
        return p.causal ? min(pos - p.cu[it.seg] + 1, seg_len) : seg_len;
    }
    if (p.remote_only) {                               // what lies before the row's own segment
        const int before = p.cu[it.seg];
        return it.kvp ? count_le_warp(it.kvp, T, before - 1, lane) : min(before, T);
    }
    if (!p.causal) return T;
    if (!it.kvp) return min(pos + 1, T);
    return count_le_warp(it.kvp, T, pos, lane);
}

// Called by a converged warp (all lanes get the same item).  kSpecial: the kernel instance that also
// serves explicit positions and bidirectional remote-only attention (two key ranges); the plain instance
// carries none of their state.  Causal remote-only attention is one more prefix mask: plain instance.
template <bool kSpecial>
__device__ __forceinline__ Item decode_item(const KernelParams &kp, int item, int lane)
{
    const PrefillParams &p = kp.p;
    Item it;
    // divisions by launch constants go through host-computed reciprocals (kp.magic_*): this runs once
    // per item in every role, on the softmax threads' critical path
    const int g = kp.group;
    const int ppg = (g + 1) >> 1;                               // head pairs per KV head
    const int per_tile = p.hkv * ppg;
    const int tile_rank = fast_div(item, kp.magic_per_tile);
    const int rem = item - tile_rank * per_tile;
    it.kvh = fast_div(rem, kp.magic_ppg);
    const int pair = rem - it.kvh * ppg;
    it.head0 = it.kvh * g + 2 * pair;
    it.valid1 = 2 * pair + 1 < g;
    // Heavy tiles first: query tiles are ranked by their index inside their segment, descending
    // (a causal tile's KV-tile count is that index + 1).  Level lv holds tile lv-1 of every segment
    // that has at least lv tiles.  With the segments sorted by tile count (ord_nt, descending), the
    // levels ord_nt[b+1] < lv <= ord_nt[b] form band b, in which every level holds the b+1 longest
    // segments; band_rank[b] = number of tiles above band b (host-computed).
    int b = 0;
    while (b + 1 < p.n_seg && tile_rank >= kp.band_rank[b + 1]) ++b;
    const int in_band = tile_rank - kp.band_rank[b];
    const int down = fast_div(in_band, kp.magic_small[b]);      // in_band / (b + 1): levels below the band's top
    const int lo = kp.ord_nt[b] - down;
    const int seg = kp.ord_seg[in_band - down * (b + 1)];
    it.seg = seg;
    it.q_row0 = p.cu[seg] + (lo - 1) * kTileM;
    it.n_valid = min(kTileM, p.cu[seg + 1] - it.q_row0);
    it.kvp = p.kv_pos ? p.kv_pos + (p.kv_head_major ? (int64_t)it.kvh * p.total_kv : 0) : nullptr;
    it.kv_begin = p.sync ? 0 : p.cu[seg];
    it.t_b0 = 0; it.a = 0; it.b = 0;
    if (kSpecial && p.general) {
        // tiles up to the last one that holds a key position <= the tile's largest query position
        const PosTables pt = pos_tables(p.tab, kp.n_qtiles, p.kv_head_major ? p.hkv : 1, kp.n_kt);
        const int32_t *suf = pt.suf_min + (p.kv_head_major ? (size_t)it.kvh * kp.n_kt : 0);
        it.n_tiles = count_le_warp(suf, kp.n_kt, __ldg(pt.q_max + (it.q_row0 >> 7)), lane);
        it.n_a = it.n_tiles;
    } else if (p.sync && p.remote_only) {
        // keys [0, a) lie before the rows' segment; when bidirectional (special instance only), keys [b, T)
        // after it count too
        const int T = (int)p.total_kv, n_t = (T + kTileN - 1) / kTileN;
        it.a = prefix_len<kSpecial>(p, it, 0, lane);
        it.n_a = (it.a + kTileN - 1) / kTileN;
        it.n_tiles = it.n_a;
        it.b = T;
        if (kSpecial && !p.causal) {
            const int after = p.cu[seg + 1];
            it.b = it.kvp ? count_le_warp(it.kvp, T, after - 1, lane) : min(after, T);
            it.t_b0 = it.b >= T ? n_t : max(it.b / kTileN, it.n_a);
            it.n_tiles = it.n_a + (n_t - it.t_b0);
        }
    } else {
        it.n_tiles = (prefix_len<kSpecial>(p, it, it.n_valid - 1, lane) + kTileN - 1) / kTileN;
        it.n_a = it.n_tiles;
    }
    return it;
}

// Persistent kernel: one CTA per SM walks the work items item = blockIdx.x, blockIdx.x + gridDim.x, ...
// Barrier phases run on: per-CTA counters of KV tiles (git) and of non-empty items (qn) give stages
// and parities, so the producer prefetches the next item's K/V and Q while the current item's last
// tiles and its epilogue are still in flight.
template <bool kSpecial>
__global__ void __launch_bounds__(kThreads, 1)
prefill_sm100_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                     const __grid_constant__ KernelParams kp)
{
    extern __shared__ uint8_t smem_raw[];
    const PrefillParams &p = kp.p;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem;                                  // [2 sub-tiles][32 KB]
    uint8_t *sK = smem + 2 * kTileBytes;                 // [2 stages][32 KB]
    uint8_t *sV = smem + 4 * kTileBytes;                 // [2 stages][32 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 6 * kTileBytes);
    uint64_t *q_full = bars + 0, *q_empty = bars + 1;
    uint64_t *k_full = bars + 2, *k_empty = bars + 4, *v_full = bars + 6, *v_empty = bars + 8;
    uint64_t *s_full = bars + 10, *o_done = bars + 12, *o_free = bars + 14;
    uint64_t *p_full = bars + 16;                        // [sub-tile][column part]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 24);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 25);
    // what the producer tells the MMA issuer about an item, published before the item's Q load is issued
    // and read after q_full: {KV tiles, sub-tiles}; -1 tiles = no more items.  Two slots, like the phases.
    volatile int *item_info = reinterpret_cast<volatile int *>(bars + 26);
    // The producer decodes every work item once and publishes it here for the softmax warps (two slots of
    // 16 ints, filled an item ahead), so that decoding is not on their path between two items.
    uint64_t *item_full = bars + 20, *item_empty = bars + 22;
    volatile int *item_pub = reinterpret_cast<volatile int *>(bars + 32);
    uint8_t *stage = smem + 6 * kTileBytes + 1024;       // [softmax warp][32 rows][128 B], 128-byte swizzle

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_items = kp.n_items;
    // Static schedule: round k hands item k*G + c to CTA c, in reversed CTA order on odd rounds, so
    // that with items sorted by cost every CTA gets a similar total.
    auto item_of = [&](int k) -> int {
        const int c = (k & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
        return k * (int)gridDim.x + c;
    };

    // ---- setup ------------------------------------------------------------------------------------
    if (tid == 0) {
        mbar_init(q_full, 1); mbar_init(q_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1);
            mbar_init(s_full + i, 1); mbar_init(o_done + i, 1); mbar_init(o_free + i, 4);
            for (int q = 0; q < kSplit; ++q) mbar_init(p_full + kSplit * i + q, 4);
            mbar_init(item_full + i, 1); mbar_init(item_empty + i, 2 * kSplit * 2);
        }
        *abort_flag = (*reinterpret_cast<volatile int32_t *>(kp.status) == FEDATTN_ERR_TIMEOUT) ? 1 : 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // A timeout that an earlier kernel reported and nobody has polled yet: this launch does no work
    // (every wait would run out again) and leaves its outputs untouched.
    const int n_rounds = *abort_flag ? 0 : (n_items + (int)gridDim.x - 1) / (int)gridDim.x;

    // every warp of a warpgroup executes the same setmaxnreg (first thing in its role); the increase
    // waits for the decrease
    if (warp == kProducerWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
        // ================= TMA producer =================
        // The whole warp decodes the work items (their searches are warp-cooperative); lane 0 waits and
        // issues the copies.
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_q) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_k) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_v) : "memory");
        }
        int git = 0, qn = 0, pn = 0;
        for (int k = 0; k < n_rounds; ++k) {
            const int item = item_of(k);
            if (item >= n_items) continue;
            const Item it = decode_item<kSpecial>(kp, item, lane);
            if (lane == 0) {
                if (pn >= 2) mbar_wait_call(item_empty + (pn & 1), ((pn >> 1) - 1) & 1, abort_flag, kp.status);
                volatile int *slot = item_pub + (pn & 1) * 16;
                slot[0] = it.kvh; slot[1] = it.head0; slot[2] = it.q_row0; slot[3] = it.n_valid; slot[4] = it.seg;
                slot[5] = it.kv_begin; slot[6] = it.n_tiles; slot[7] = it.n_a; slot[8] = it.t_b0; slot[9] = it.a;
                slot[10] = it.b; slot[11] = it.valid1 ? 1 : 0;
                mbar_arrive(item_full + (pn & 1));
                if (it.n_tiles > 0) {
                    // this item's Q on its way into L2: the load itself has to wait for the Q buffer
                    tma_prefetch_3d(&map_q, 0, it.head0, it.q_row0);
                    tma_prefetch_3d(&map_q, 64, it.head0, it.q_row0);
                    if (it.valid1) {
                        tma_prefetch_3d(&map_q, 0, it.head0 + 1, it.q_row0);
                        tma_prefetch_3d(&map_q, 64, it.head0 + 1, it.q_row0);
                    }
                }
            }
            ++pn;
            if (it.n_tiles == 0) continue;
            if (lane == 0) {
                if (qn > 0) mbar_wait_call(q_empty, (qn - 1) & 1, abort_flag, kp.status);   // previous item's S MMAs done
                item_info[(qn & 1) * 2] = it.n_tiles;
                item_info[(qn & 1) * 2 + 1] = it.valid1 ? 2 : 1;
                mbar_expect_tx(q_full, it.valid1 ? 2 * kTileBytes : kTileBytes);
                tma_load_3d(sQ, &map_q, q_full, 0, it.head0, it.q_row0);
                tma_load_3d(sQ + kHalfBytes, &map_q, q_full, 64, it.head0, it.q_row0);
                if (it.valid1) {
                    tma_load_3d(sQ + kTileBytes, &map_q, q_full, 0, it.head0 + 1, it.q_row0);
                    tma_load_3d(sQ + kTileBytes + kHalfBytes, &map_q, q_full, 64, it.head0 + 1, it.q_row0);
                }
                for (int j = 0; j < it.n_tiles; ++j) {
                    const int gt = git + j, st = gt & 1, use = gt >> 1;
                    const int row = it.kv_begin + (kSpecial ? tile_of(it, j) : j) * kTileN;
                    const int c1 = p.kv_head_major ? row : it.kvh, c2 = p.kv_head_major ? it.kvh : row;
                    if (gt >= 2) mbar_wait_call(k_empty + st, (use - 1) & 1, abort_flag, kp.status);
                    TRACE(j, 7);
                    mbar_expect_tx(k_full + st, kTileBytes);
                    tma_load_3d(sK + st * kTileBytes, &map_k, k_full + st, 0, c1, c2);
                    tma_load_3d(sK + st * kTileBytes + kHalfBytes, &map_k, k_full + st, 64, c1, c2);
                    if (gt >= 2) mbar_wait_call(v_empty + st, (use - 1) & 1, abort_flag, kp.status);
                    mbar_expect_tx(v_full + st, kTileBytes);
                    tma_load_3d(sV + st * kTileBytes, &map_v, v_full + st, 0, c1, c2);
                    tma_load_3d(sV + st * kTileBytes + kHalfBytes, &map_v, v_full + st, 64, c1, c2);
                }
            }
            __syncwarp();
            git += it.n_tiles;
            ++qn;
        }
        if (lane == 0) {
            // end marker for the MMA issuer, in the slot and phase the next item would have used
            if (qn > 0) mbar_wait_call(q_empty, (qn - 1) & 1, abort_flag, kp.status);
            item_info[(qn & 1) * 2] = -1;
            mbar_arrive(q_full);
            if (*abort_flag) {
                // give the copies still in flight a bounded chance to land before the CTA retires
                for (int gt = max(0, git - 2); gt < git; ++gt) {
                    for (uint32_t w = 0; w < 4096 && !mbar_try_wait(k_full + (gt & 1), (gt >> 1) & 1); ++w) {}
                    for (uint32_t w = 0; w < 4096 && !mbar_try_wait(v_full + (gt & 1), (gt >> 1) & 1); ++w) {}
                }
                if (qn > 0)
                    for (uint32_t w = 0; w < 4096 && !mbar_try_wait(q_full, (qn - 1) & 1); ++w) {}
            }
        }
    } else if (warp == kMmaWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
        // ================= MMA issuer =================
        // Issue order per item  S0(0) S1(0) | PV0(0) S0(1) | PV1(0) S1(1) | PV0(1) S0(2) | ...  : while one
        // sub-tile's softmax runs, the tensor pipe works on the other sub-tile.
        // The whole warp walks the loop (waits included) so that control flow and operand descriptors
        // stay warp-uniform; one elected lane issues the tcgen05 instructions.  Issued from inside a
        // single-lane branch the same instructions sustain only ~83 cycles per MMA instead of 64.
        const bool leader = elect_one();
        const uint32_t aQ = smem_u32(sQ), aK = smem_u32(sK), aV = smem_u32(sV);
        const uint64_t dQ = make_desc(aQ, 16, 1024), dK = make_desc(aK, 16, 1024), dV = make_desc(aV, kHalfBytes, 1024);
        auto issue_s = [&](int t, int st) {
            if (leader) {
#pragma unroll
                for (int ks = 0; ks < kD / 16; ++ks) {
                    const uint32_t off = ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;       // descriptor units
                    umma_ss(tmem_base + kColS + t * 128, dQ + (uint64_t)(t * (kTileBytes >> 4) + off),
                            dK + (uint64_t)(st * (kTileBytes >> 4) + off), kIdescQK, ks > 0);
                }
            }
        };
        auto commit = [&](uint64_t *bar) { if (leader) tc_commit(bar); };
        // git / qn count the KV tiles / items of sub-tile 0 (and of the K/V ring); git1 / qn1
        // count only the items in which the pair's second head exists.
        int git = 0, qn = 0, git1 = 0, qn1 = 0;
        for (;;) {
            // the producer decodes the work items; this warp only learns their shape (decoding them here as
            // well does not fit into this role's 64 registers)
            if (!mbar_wait_call(q_full, qn & 1, abort_flag, kp.status)) break;
            const int n = item_info[(qn & 1) * 2];
            if (n < 0) break;
            const int n_sub = item_info[(qn & 1) * 2 + 1];
            mbar_wait_call(k_full + (git & 1), (git >> 1) & 1, abort_flag, kp.status);
            tc_fence_after();
            for (int t = 0; t < n_sub; ++t) {
                issue_s(t, git & 1);
                commit(s_full + t);
            }
            commit(k_empty + (git & 1));
            if (n == 1) commit(q_empty);
            for (int j = 0; j < n; ++j) {
                const int gt = git + j, st = gt & 1, ph = (gt >> 1) & 1;
                const int st1 = (gt + 1) & 1, ph1 = ((gt + 1) >> 1) & 1;
                for (int t = 0; t < n_sub; ++t) {
                    const int gsub = (t ? git1 : git) + j, qsub = t ? qn1 : qn;
                    if (t == 0) mbar_wait_call(v_full + st, ph, abort_flag, kp.status);
                    if (j == 0 && qsub > 0) mbar_wait_call(o_free + t, (qsub - 1) & 1, abort_flag, kp.status);
#pragma unroll
                    for (int q = 0; q < kSplit; ++q) {
                        mbar_wait_call(p_full + kSplit * t + q, gsub & 1, abort_flag, kp.status);
                        if (lane == 0 && q == 0) TRACE(j, 2 + t);
                        tc_fence_after();
                        if (leader) {
#pragma unroll
                            for (int kk = 0; kk < kCols / 16; ++kk) {
                                const int ks = q * (kCols / 16) + kk;
                                umma_ts(tmem_base + kColO + t * 128, tmem_base + kColS + t * 128 + q * kCols + kk * 8,
                                        dV + (uint64_t)(st * (kTileBytes >> 4) + ks * (2048 >> 4)), kIdescPV,
                                        (j > 0 || ks > 0));
                            }
                        }
                    }
                    commit(o_done + t);
                    if (t == n_sub - 1) commit(v_empty + st);
                    if (j + 1 < n) {
                        if (t == 0) mbar_wait_call(k_full + st1, ph1, abort_flag, kp.status);
                        issue_s(t, st1);
                        commit(s_full + t);
                        if (t == n_sub - 1) {
                            commit(k_empty + st1);
                            if (j + 2 == n) commit(q_empty);     // last S of this item issued
                        }
                    }
                    if (t == 1 && lane == 0) TRACE(j, 4);
                }
            }
            git += n;
            ++qn;
            if (n_sub == 2) { git1 += n; ++qn1; }
        }
    } else if (warp >= 4 * kSplit) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));      // the two idle warps of that warpgroup
        // One of them checks what the prefix-count mask relies on: key positions that never decrease
        // along the aggregated rows of a head.  The CTAs share the pairs (i, i + 1) among them.
        if (warp == kMmaWarp + 1 && p.kv_pos && !p.general && p.sync && (p.causal || p.remote_only) && p.total_kv > 1) {
            const int64_t per = p.total_kv - 1, total = per * (p.kv_head_major ? p.hkv : 1);
            bool bad = false;
            for (int64_t i = (int64_t)blockIdx.x * 32 + lane; i < total; i += (int64_t)gridDim.x * 32) {
                const int64_t a = i / per, e = a * p.total_kv + (i - a * per);
                bad |= __ldg(p.kv_pos + e) > __ldg(p.kv_pos + e + 1);
            }
            if (bad) atomicMax(kp.status, (int32_t)FEDATTN_ERR_ORDER);
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
        // ================= softmax + epilogue =================
        // Warpgroup t serves sub-tile t (query head head0 + t) on its own: thread = query row r = TMEM lane,
        // all 128 key columns of the S tile, the whole row of O.  The two warpgroups never meet: no row
        // maximum or row sum has to be exchanged, and while one is in the serial part of its visit (wait,
        // TMEM load, maximum) the other computes.  A thread reads its row of S from TMEM once and keeps all
        // 128 values in registers for both walks (maximum, then exponentials).
        const int t = warp >> 2;                                // sub-tile of this warpgroup
        const int r = tid & 127;                                // query row = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_base + kColS + t * 128;   // fp32 S; bf16 P of keys 64q.. at column 64q
        const uint32_t tO = tmem_base + lane_base + kColO + t * 128;
        const float sl2 = p.scale * 1.4426950408889634f;
        const uint64_t sl2_2 = pack_f32x2(sl2, sl2);
        int gsub = 0;                                           // KV tiles this sub-tile has been through
        auto below32 = [](int n) -> uint32_t { return n <= 0 ? 0u : (n >= 32 ? 0xffffffffu : (1u << n) - 1u); };

        // One visit = the softmax of one S tile.  kPartial: some row of the tile has masked columns; bit i of
        // vm[c] says whether column 32 c + i is visible to this thread's row.  Masked columns become -inf and
        // every exponential goes through ex2.approx, which maps -inf to 0; in unmasked tiles a fixed subset of
        // the columns takes the polynomial so that the ex2 unit is not the bottleneck.
        auto visit = [&](auto partial_tag, int j, int gt, const uint32_t (&vm)[4], float &m_used, float &l) {
            constexpr bool kPartial = decltype(partial_tag)::value;
            mbar_wait(s_full + t, gt & 1, abort_flag, kp.status);
            if (tid == 0) TRACE(j, t ? 5 : 0);
            tc_fence_after();
            // the whole row of S in registers: read from TMEM once, used for the maximum and the exponentials
            uint32_t s0[32], s1[32], s2[32], s3[32];
            float mx[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
            FEDATTN_TMEM_LD32(tS, s0);
            FEDATTN_TMEM_LD32(tS + 32, s1);
            tmem_wait_ld();
            FEDATTN_TMEM_LD32(tS + 64, s2);
            FEDATTN_TMEM_LD32(tS + 96, s3);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t *cur = c == 0 ? s0 : (c == 1 ? s1 : (c == 2 ? s2 : s3));
                if (c == 2) tmem_wait_ld();
                if (kPartial) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (!((vm[c] >> i) & 1u)) cur[i] = 0xff800000u;          // -inf
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    mx[i] = max3(mx[i], __uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1]));
                    mx[i] = max3(mx[i], __uint_as_float(cur[16 + 2 * i]), __uint_as_float(cur[16 + 2 * i + 1]));
                }
            }
            const float rm = fmaxf(max3(mx[0], mx[1], mx[2]), fmaxf(max3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
            const float t_max = rm * sl2;
            if (j == 0) {
                m_used = (t_max == -INFINITY) ? 0.f : t_max;
            } else {
                // The exponent reference moves only when the maximum grew by more than 2^8; then what
                // this row has accumulated so far (O in TMEM, l) is rescaled to the new reference.
                const bool need = t_max > m_used + kRescaleThreshold;
                if (__any_sync(0xffffffffu, need)) {
                    const float alpha = need ? ex2(m_used - t_max) : 1.f;
                    mbar_wait(o_done + t, (gt - 1) & 1, abort_flag, kp.status);   // O holds tiles 0..j-1
                    tc_fence_after();
#pragma unroll 1
                    for (int oc = 0; oc < 4; ++oc) {
                        uint32_t o[32];
                        FEDATTN_TMEM_LD32(tO + oc * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        FEDATTN_TMEM_ST32(tO + oc * 32, o);
                    }
                    if (need) { l *= alpha; m_used = t_max; }
                }
            }
            // ---- pass 2: exponentials, row sum, P ----
            const uint64_t negm2 = pack_f32x2(-m_used, -m_used);
            uint64_t sum2[4] = {0, 0, 0, 0};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t *cur = c == 0 ? s0 : (c == 1 ? s1 : (c == 2 ? s2 : s3));
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1])), sl2_2, negm2);
                    float p0, p1;
                    if (!kPartial && ((kPolyMask >> (i & 7)) & 1)) {
                        exp2_poly_x2(x2, p0, p1);
                    } else {
                        float x0, x1;
                        unpack_f32x2(x2, x0, x1);
                        p0 = ex2(x0); p1 = ex2(x1);
                    }
                    sum2[i & 3] = add_f32x2(sum2[i & 3], pack_f32x2(p0, p1));
                    pk[i] = pack_bf16(p0, p1);
                }
                // keys 32 c .. 32 c + 31 as bf16 pairs: columns 64 (c / 2) + 16 (c % 2) .., all inside S columns
                // that this thread has already read
                FEDATTN_TMEM_ST16(tS + 64 * (c >> 1) + 16 * (c & 1), pk);
                if (c & 1) {                                    // a 64-key half of P is complete: PV may start on it
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(p_full + kSplit * t + (c >> 1));      // one arrival per warp
                }
            }
            float r0, r1;
            unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), r0, r1);
            l += r0 + r1;
            if (tid == 0) TRACE(j, t ? 6 : 1);
        };

        int pn = 0;                                             // items read from the producer's slots
        for (int k = 0; k < n_rounds; ++k) {
            const int item = item_of(k);
            if (item >= n_items) continue;
            Item it;
            {
                mbar_wait(item_full + (pn & 1), (pn >> 1) & 1, abort_flag, kp.status);
                const volatile int *slot = item_pub + (pn & 1) * 16;
                it.kvh = slot[0]; it.head0 = slot[1]; it.q_row0 = slot[2]; it.n_valid = slot[3]; it.seg = slot[4];
                it.kv_begin = slot[5]; it.n_tiles = slot[6]; it.n_a = slot[7]; it.t_b0 = slot[8]; it.a = slot[9];
                it.b = slot[10]; it.valid1 = slot[11] != 0;
                it.kvp = p.kv_pos ? p.kv_pos + (p.kv_head_major ? (int64_t)it.kvh * p.total_kv : 0) : nullptr;
                __syncwarp();
                if (lane == 0) mbar_arrive(item_empty + (pn & 1));
                ++pn;
            }
            if (t == 1 && !it.valid1) continue;                 // the pair's second head does not exist
            const int n_tiles = it.n_tiles;
            const bool valid = r < it.n_valid;
            __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(p.o) + ((int64_t)(it.q_row0 + r) * p.hq + it.head0 + t) * kD;
            float *lse_p = p.lse ? p.lse + (int64_t)(it.q_row0 + r) * p.hq + it.head0 + t : nullptr;
            if (n_tiles == 0) {                                 // nothing visible to any row of the tile
                if (valid) {
#pragma unroll
                    for (int c = 0; c < kD; c += 8) *reinterpret_cast<uint4 *>(orow + c) = make_uint4(0, 0, 0, 0);
                    if (lse_p) *lse_p = -INFINITY;
                }
                continue;
            }
            const bool two_range = kSpecial && p.sync && p.remote_only && !p.causal;
            const bool general = kSpecial && p.general;
            int c_row = 0, n_full = 0, p_row = 0;
            if (general) {
                // every (query, key) pair on its own positions; the tiles whose keys all lie at or below the
                // tile's smallest query position (a prefix of the walk, see PosTables) need no test
                const PosTables pt = pos_tables(p.tab, kp.n_qtiles, p.kv_head_major ? p.hkv : 1, kp.n_kt);
                const int32_t *pre = pt.pre_max + (p.kv_head_major ? (size_t)it.kvh * kp.n_kt : 0);
                n_full = count_le_warp(pre, kp.n_kt, __ldg(pt.q_min + (it.q_row0 >> 7)), lane);
                const int row = it.q_row0 + min(r, it.n_valid - 1);
                p_row = p.q_pos ? __ldg(p.q_pos + row) : row;
            } else {
                if (p.sync && p.remote_only) {
                    c_row = it.a;                               // the same for every row of the segment
                } else if (p.sync && p.causal && it.kvp) {
                    // Sparse aggregate, row position = row index.  One cooperative search gives the keys
                    // visible to all of the warp's 32 consecutive rows; the next 32 keys are the only ones
                    // that can tell these rows apart (more only if positions repeat: then each lane searches).
                    const int T = (int)p.total_kv, p0 = it.q_row0 + (r & ~31);
                    const int cw = count_le_warp(it.kvp, T, p0 - 1, lane);
                    const int wv = cw + lane < T ? __ldg(it.kvp + cw + lane) : INT32_MAX;
                    int cnt = 0;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) cnt += __shfl_sync(0xffffffffu, wv, jj) <= p0 + lane;
                    c_row = cw + cnt;
                    if (__shfl_sync(0xffffffffu, wv, 31) <= p0 + 31) c_row = count_le(it.kvp, T, p0 + lane);
                } else {
                    c_row = prefix_len<kSpecial>(p, it, r, lane);   // arithmetic only
                }
                // prefix lengths do not decrease with the row, so KV tiles below the prefix of the warp's first
                // row are unmasked for the whole warp (the choice of code path only has to be warp-uniform)
                n_full = __shfl_sync(0xffffffffu, c_row, 0) / kTileN;
            }
            const int T = (int)p.total_kv;
            float m_run = 0.f, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j) {
                const int gt = gsub + j;
                // which columns of this tile the thread's row sees: everything (warp-uniform), or a mask per chunk
                bool full;
                uint32_t vm[4] = {0, 0, 0, 0};
                if (two_range) {                                // keys [0, a) and [b, T)
                    const int k0 = tile_of(it, j) * kTileN;     // first key of the tile
                    full = k0 + kTileN <= it.a || (k0 >= it.b && k0 + kTileN <= T);
                    if (!full) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int cb = k0 + 32 * c;
                            vm[c] = below32(it.a - cb) | (below32(T - cb) & ~below32(it.b - cb));
                        }
                    }
                } else {
                    full = j < n_full;
                    if (!full && general) {
                        // column i of chunk c is key cb + i: visible iff it exists and its position is not above
                        // the row's.  The address is the same in every lane: broadcast loads.
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int cb = j * kTileN + 32 * c;
                            uint32_t m = 0;
#pragma unroll 4
                            for (int i = 0; i < 32; ++i) {
                                const int key = cb + i;
                                const int kpos = it.kvp ? __ldg(it.kvp + min(key, T - 1)) : key;
                                if (key < T && kpos <= p_row) m |= 1u << i;
                            }
                            vm[c] = m;
                        }
                    } else if (!full) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) vm[c] = below32(c_row - j * kTileN - 32 * c);
                    }
                }
                if (full) visit(std::false_type{}, j, gt, vm, m_run, l_run);
                else visit(std::true_type{}, j, gt, vm, m_run, l_run);
            }

            // ---- epilogue: drain this row of O from TMEM (frees it for the next item), O / l -> bf16 -> global
            mbar_wait(o_done + t, (gsub + n_tiles - 1) & 1, abort_flag, kp.status);
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            // Full warps of rows leave through shared memory and TMA stores (a warp's 32 rows x 64 columns at a
            // time); a warp with rows beyond the segment writes its valid rows directly.
            const bool by_tma = kp.o_tma && (r | 31) < it.n_valid;
            uint8_t *my_stage = stage + (size_t)warp * kStageBytes;
            if (by_tma) {
                if (lane == 0) tma_store_wait_read();           // the previous item's last store has read the staging rows
                __syncwarp();
                uint32_t oa[32], ob[32];
                FEDATTN_TMEM_LD32(tO, oa);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t *cur = (c & 1) ? ob : oa, *nxt = (c & 1) ? oa : ob;
                    tmem_wait_ld();
                    if (c < 3) {
                        FEDATTN_TMEM_LD32(tO + 32 * (c + 1), nxt);
                    } else {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(o_free + t); // one arrival per warp: O_t may be overwritten
                    }
                    if (c == 2) {                               // the first half's store has read the staging rows
                        if (lane == 0) tma_store_wait_read();
                        __syncwarp();
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {               // 16-byte unit 4 (c & 1) + u of the row's 128 staged bytes
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            w[i] = pack_bf16(__uint_as_float(cur[8 * u + 2 * i]) * inv, __uint_as_float(cur[8 * u + 2 * i + 1]) * inv);
                        const int unit = 4 * (c & 1) + u;
                        *reinterpret_cast<uint4 *>(my_stage + lane * 128 + ((unit ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (c & 1) {
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) tma_store_3d(&map_o, my_stage, 64 * (c >> 1), it.head0 + t, it.q_row0 + (r & ~31));
                    }
                }
            } else {
                // the rare path (a warp with rows beyond the segment) is kept short rather than fast
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    FEDATTN_TMEM_LD32(tO + 32 * c, o);
                    tmem_wait_ld();
                    if (c == 3) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(o_free + t);
                    }
                    if (valid) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            uint32_t w[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                w[i] = pack_bf16(__uint_as_float(o[8 * u + 2 * i]) * inv, __uint_as_float(o[8 * u + 2 * i + 1]) * inv);
                            *reinterpret_cast<uint4 *>(orow + 32 * c + 8 * u) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
            if (valid && lse_p) *lse_p = l_run > 0.f ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            gsub += n_tiles;
        }
        if (lane == 0) tma_store_wait_read();                   // the staging rows stay alive until they are read
    }

    // ---- teardown -----------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarp) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- position tables of a general-position call -------------------------------------------------------
// grid: one block per KV position array (n_arrays of them), then one block for the query positions.
// A warp reduces one 128-entry tile at a time (one 16-byte load per lane when the array allows it).  The
// KV blocks then turn the per-tile values into the running suffix minimum / prefix maximum in place.
constexpr int kTabThreads = 1024;

__device__ __forceinline__ void tile_min_max(const int32_t *pos, int64_t n, int64_t tile, int lane, int &mn, int &mx)
{
    mn = INT32_MAX; mx = INT32_MIN;
    const int64_t i0 = tile * kTileN + lane * 4;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int64_t i = i0 + e;
        if (i < n) {
            const int v = pos ? __ldg(pos + i) : (int)i;
            mn = min(mn, v); mx = max(mx, v);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
}

__global__ void __launch_bounds__(kTabThreads)
position_tables_kernel(const int32_t *q_pos, int64_t n_q, const int32_t *kv_pos, int64_t total_kv, int n_arrays,
                       int n_qtiles, int n_kt, int32_t *tab)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = kTabThreads / 32;
    const PosTables pt = pos_tables(tab, n_qtiles, n_arrays, n_kt);
    if ((int)blockIdx.x == n_arrays) {
        int32_t *q_min = tab, *q_max = tab + n_qtiles;
        for (int64_t t = warp; t < n_qtiles; t += n_warps) {
            int mn, mx;
            tile_min_max(q_pos, n_q, t, lane, mn, mx);
            if (lane == 0) { q_min[t] = mn; q_max[t] = mx; }
        }
        return;
    }
    const int a = blockIdx.x;
    const int32_t *pos = kv_pos ? kv_pos + (size_t)a * total_kv : nullptr;
    int32_t *suf = const_cast<int32_t *>(pt.suf_min) + (size_t)a * n_kt, *pre = const_cast<int32_t *>(pt.pre_max) + (size_t)a * n_kt;
    for (int64_t t = warp; t < n_kt; t += n_warps) {
        int mn, mx;
        tile_min_max(pos, total_kv, t, lane, mn, mx);
        if ((t + 1) * kTileN > total_kv) mx = INT32_MAX;      // ragged tile: never fully visible
        if (lane == 0) { suf[t] = mn; pre[t] = mx; }
    }
    __syncthreads();
    if (warp == 0) {                                           // prefix maximum, 32 tiles per step
        int carry = INT32_MIN;
        for (int t0 = 0; t0 < n_kt; t0 += 32) {
            int v = t0 + lane < n_kt ? pre[t0 + lane] : INT32_MIN;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v = max(v, u);
            }
            v = max(v, carry);
            if (t0 + lane < n_kt) pre[t0 + lane] = v;
            carry = __shfl_sync(0xffffffffu, v, 31);
        }
    } else if (warp == 1) {                                    // suffix minimum, from the last tile backwards
        int carry = INT32_MAX;
        for (int t0 = ((n_kt - 1) / 32) * 32; t0 >= 0; t0 -= 32) {
            int v = t0 + lane < n_kt ? suf[t0 + lane] : INT32_MAX;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_down_sync(0xffffffffu, v, o);
                if (lane + o < 32) v = min(v, u);
            }
            v = min(v, carry);
            if (t0 + lane < n_kt) suf[t0 + lane] = v;
            carry = __shfl_sync(0xffffffffu, v, 0);
        }
    }
}

// ---- self-test of the bounded wait ---------------------------------------------------------------------
// Waits with mbar_wait, the routine every role above waits with, on a barrier that nothing signals.
__global__ void wait_selftest_kernel(int32_t *status, uint32_t max_polls)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_flag, status, max_polls);        // phase 0 never completes: runs out, flags the status
}

// ---- host ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

#ifdef FEDATTN_TRACE
extern "C" int fedattn_debug_read_trace(long long *host, int n)
{
    return (int)cudaMemcpyFromSymbol(host, g_trace, sizeof(long long) * n);
}
#endif

bool prefill_sm100_supported(const Context *ctx) { return ctx->encode_tiled != nullptr; }

// [rows, heads, 128] bf16 (token-major) or [heads, rows, 128] (head-major); boxes of 64 columns x 128 rows.
static bool encode_map(const Context *ctx, CUtensorMap *map, const void *base, int64_t rows, int heads, bool head_major,
                       int box_rows = kTileN)
{
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t dims[3], strides[2];
    cuuint32_t box[3], estr[3] = {1, 1, 1};
    dims[0] = kD;
    if (head_major) {
        dims[1] = (cuuint64_t)rows; dims[2] = (cuuint64_t)heads;
        strides[0] = kD * 2; strides[1] = (cuuint64_t)rows * kD * 2;
        box[0] = 64; box[1] = (cuuint32_t)box_rows; box[2] = 1;
    } else {
        dims[1] = (cuuint64_t)heads; dims[2] = (cuuint64_t)rows;
        strides[0] = kD * 2; strides[1] = (cuuint64_t)heads * kD * 2;
        box[0] = 64; box[1] = 1; box[2] = (cuuint32_t)box_rows;
    }
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t position_table_bytes(int hkv, int64_t n_q_rows, int64_t total_kv)
{
    const int64_t n_qt = (n_q_rows + kTileM - 1) / kTileM, n_kt = (total_kv + kTileN - 1) / kTileN;
    return (size_t)(2 * n_qt + 2 * (int64_t)hkv * n_kt) * sizeof(int32_t);
}

cudaError_t launch_wait_selftest(Context *ctx, int max_polls, cudaStream_t s)
{
    wait_selftest_kernel<<<1, 32, 0, s>>>(ctx->status, (uint32_t)max_polls);
    ++ctx->launches;
    return cudaGetLastError();
}

cudaError_t launch_prefill_sm100(Context *ctx, const PrefillParams &p, cudaStream_t s)
{
    static_assert(sizeof(KernelParams) < 3000, "kernel parameter block too large");
    KernelParams kp;
    kp.p = p;
    kp.status = ctx->status;
    kp.n_kt = (int32_t)((p.total_kv + kTileN - 1) / kTileN);
    int64_t n_qtiles = 0;
    for (int n = 0; n < p.n_seg; ++n) {
        kp.ord_seg[n] = n;
        kp.ord_nt[n] = (p.cu[n + 1] - p.cu[n] + kTileM - 1) / kTileM;
        n_qtiles += kp.ord_nt[n];
    }
    for (int a = 1; a < p.n_seg; ++a)          // insertion sort by tile count, descending (stable)
        for (int b = a; b > 0 && kp.ord_nt[b] > kp.ord_nt[b - 1]; --b) {
            const int32_t tn = kp.ord_nt[b], ts = kp.ord_seg[b];
            kp.ord_nt[b] = kp.ord_nt[b - 1]; kp.ord_seg[b] = kp.ord_seg[b - 1];
            kp.ord_nt[b - 1] = tn; kp.ord_seg[b - 1] = ts;
        }
    if (n_qtiles > 0x7fffffffLL) return cudaErrorInvalidValue;
    kp.band_rank[0] = 0;
    for (int b = 0; b < p.n_seg; ++b) {
        const int64_t next = b + 1 < p.n_seg ? kp.ord_nt[b + 1] : 0;
        kp.band_rank[b + 1] = kp.band_rank[b] + (int32_t)((kp.ord_nt[b] - next) * (b + 1));
    }
    kp.n_qtiles = (int32_t)n_qtiles;
    const int g = p.hq / p.hkv;
    const int64_t items = n_qtiles * p.hkv * ((g + 1) / 2);
    if (items == 0) return cudaSuccess;
    if (items >= (1LL << 28) || (int64_t)p.hkv * ((g + 1) / 2) > 4096) return cudaErrorInvalidValue;   // fast_div range
    kp.n_items = (int32_t)items;
    auto magic = [](int64_t d) { return (uint64_t)(((1ULL << 40) + (uint64_t)d - 1) / (uint64_t)d); };
    kp.group = g;
    kp.magic_per_tile = magic((int64_t)p.hkv * ((g + 1) / 2));
    kp.magic_ppg = magic((g + 1) / 2);
    for (int i = 0; i < kMaxP; ++i) kp.magic_small[i] = magic(i + 1);
    const int64_t blocks = items < ctx->sm_count ? items : ctx->sm_count;     // persistent: one CTA per SM
    CUtensorMap mq, mk, mv, mo;
    if (!encode_map(ctx, &mq, p.q, p.n_q_rows, p.hq, false) ||
        !encode_map(ctx, &mk, p.k, p.total_kv, p.hkv, p.kv_head_major != 0) ||
        !encode_map(ctx, &mv, p.v, p.total_kv, p.hkv, p.kv_head_major != 0))
        return cudaErrorInvalidValue;
    // the output as [rows, heads, 128] in boxes of 32 rows x 64 columns; a base the encoder refuses (alignment)
    // leaves the kernel on its direct stores
    kp.o_tma = encode_map(ctx, &mo, p.o, p.n_q_rows, p.hq, false, 32) ? 1 : 0;
    if (!kp.o_tma) mo = mq;
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_sm100_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(prefill_sm100_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        // the register split inside the kernel has to fit into what the launch allocates: an increase that
        // the CTA's pool cannot serve would wait for ever, so such a build is refused here
        cudaFuncAttributes fa0, fa1;
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa0, prefill_sm100_kernel<false>);
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa1, prefill_sm100_kernel<true>);
        if (e == cudaSuccess && (3 * fa0.numRegs < 2 * kSoftmaxRegs + kOtherRegs || 3 * fa1.numRegs < 2 * kSoftmaxRegs + kOtherRegs))
            e = cudaErrorLaunchOutOfResources;
        if (e != cudaSuccess) {
            if (getenv("FEDATTN_DEBUG")) fprintf(stderr, "prefill_sm100_kernel attribute: %s\n", cudaGetErrorString(e));
            return e;
        }
        attr_set[ctx->device & 63] = true;
    }
    if (p.general) {
        // the per-tile position tables first (same stream): the walk and the unmasked fast path read them
        const int n_arrays = p.kv_head_major ? p.hkv : 1;
        position_tables_kernel<<<n_arrays + 1, kTabThreads, 0, s>>>(p.q_pos, p.n_q_rows, p.kv_pos, p.total_kv, n_arrays,
                                                                    kp.n_qtiles, kp.n_kt, p.tab);
        ++ctx->launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    // the plain instance serves local attention and sync attention under the prefix mask; explicit positions
    // and remote-only attention run the instance that carries their extra state
    if (p.general || (p.remote_only && !p.causal)) prefill_sm100_kernel<true><<<(unsigned)blocks, kThreads, kSmemBytes, s>>>(mq, mk, mv, mo, kp);
    else prefill_sm100_kernel<false><<<(unsigned)blocks, kThreads, kSmemBytes, s>>>(mq, mk, mv, mo, kp);
    ++ctx->launches;
    ++ctx->tc_launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess && getenv("FEDATTN_DEBUG")) fprintf(stderr, "prefill_sm100_kernel launch: %s\n", cudaGetErrorString(e));
    return e;
}

}  // namespace fedattn
