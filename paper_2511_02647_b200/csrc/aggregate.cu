// KV aggregation kernels: dense concatenation, key-norm scores, per-(participant, head) top-k
// selection, and the indexed gather that builds the head-major sparse KV.  All are pure data
// movement or integer/compare work except the score, which is an fp64 chain in fixed order so
// that the selected set is bit-identical to a sequential fp64 evaluation.
#include <cooperative_groups.h>
#include <string.h>

#include <limits.h>

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
// s + x^2 for the two bf16 values packed in w, low half first; each square is exact in fp64.
// (Widening by integer bit moves instead of the fp32->fp64 conversion, for all or for half of the
// terms, was measured no faster: four integer instructions cost the integer pipe what one
// conversion costs the conversion unit, and the phase waits for its data more than for either.)
__device__ __forceinline__ double sq_acc_bf16x2(double s, uint32_t w)
{
    const double lo = (double)__uint_as_float(w << 16);
    const double hi = (double)__uint_as_float(w & 0xffff0000u);
    // x * x is exact in fp64, so the fused multiply-add rounds exactly once, like the separate add
    s = __fma_rn(lo, lo, s);
    s = __fma_rn(hi, hi, s);
    return s;
}

// ---- top-k scores + selection + gather, one launch ----------------------------------------------
// grid (KV head, participant, slice); the slices of one (head, participant) form a thread-block
// cluster.
//  1. Scores.  Slice r takes a contiguous share of the participant's tokens.  Every warp copies the K
//     rows of this head for 32 tokens at a time (row_bytes each, strided by the token pitch) into a
//     ring of its own in shared memory with 16-byte cp.async, 128 bytes of every row per step, and
//     lane i walks row i: s = sum_c x_c^2 accumulated in fp64 in increasing c.  Each square of a
//     bf16/fp32 value is exact in fp64, so only the order matters and it is fixed.  Scores are
//     non-negative doubles, so their bit patterns order like unsigned integers; they are kept as such
//     keys in shared memory.
//  2. Every slice collects the other slices' keys through distributed shared memory.
//  3. Selection, repeated by every slice: an 8-bit-per-pass radix select, started at the highest bit
//     in which two keys differ, finds the k-th largest score tau and how many rows equal to tau are
//     still needed; the keys of the first chosen bin are listed and, when the list is short, ranked
//     by counting instead of further passes.  One ordered compaction then gives every kept row its
//     output position (rows with score > tau, plus the lowest-index rows with score == tau, in
//     ascending index order).
//  4. Slice r copies its share of the kept K/V rows into the head-major output and writes their
//     indices and global positions.
constexpr int kSelThreads = 256;
constexpr int kSelMaxLen = 4096;
constexpr int kMaxSlices = 8;              // portable cluster size
constexpr int kCtasPerSm = 2;              // resident CTAs the staging rings are sized for

template <int kDtype>
__global__ void __launch_bounds__(kSelThreads)
topk_fused_kernel(const PartsParams pp, int hkv, int vpr /* 16-byte vectors per (row, head) */,
                  int n_stages /* buffers in every warp's staging ring, 2..4 */,
                  int max_len /* longest participant: sizes the key arrays */,
                  int early /* the inputs may be read before the preceding grid of the stream is complete */,
                  long long my_seq /* this call's sequence number in its context */,
                  long long need_seq /* the latest call that writes one of this call's outputs (0: none) */,
                  long long *done_seq /* the context's word: largest sequence number known to be complete */,
                  uint4 *k_agg, uint4 *v_agg, int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out)
{
    // dynamic shared memory: keys [max_len] u64 | kept rows [max_len] u16 | staging [8 warps][n_stages][32 rows][128 B]
    extern __shared__ __align__(16) uint8_t dyn_smem[];
    unsigned long long *keys = reinterpret_cast<unsigned long long *>(dyn_smem);
    uint16_t *my_rows = reinterpret_cast<uint16_t *>(dyn_smem + (size_t)max_len * 8);   // kept indices of this CTA's slice (< 4096)
    uint8_t *stage = dyn_smem + (((size_t)max_len * 10 + 15) & ~(size_t)15);
    __shared__ int hist[256];
    __shared__ int warp_tot[kSelThreads / 32];
    __shared__ int sh_bin, sh_krem, sh_count;
    __shared__ unsigned long long sh_tau;
    __shared__ unsigned long long warp_or[kSelThreads / 32], warp_and[kSelThreads / 32];

    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int h = blockIdx.x, n = blockIdx.y, slice = blockIdx.z, n_slices = gridDim.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Launched with programmatic stream serialization: the dependents may take their seats at once.
    // Inputs are read before the preceding grid of the stream is known to be complete unless they might be
    // its outputs (early == 0).  Outputs are written at once when every earlier call that writes the same
    // buffers is known to be over (*done_seq >= need_seq), else after griddepcontrol.wait.  One CTA of the
    // grid always waits for the preceding grid before it exits: a grid must not complete before its
    // predecessor, or what follows in the stream could overtake earlier work; that CTA then records that
    // every call before this one is complete.
    if (!early) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool closer = h == 0 && n == 0 && slice == 0;
    auto close_call = [&]() {
        if (closer) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (tid == 0 && my_seq > 0) atomicMax(reinterpret_cast<unsigned long long *>(done_seq), (unsigned long long)(my_seq - 1));
        }
    };
    // The call it has to see complete is an EARLIER grid of the stream, all of whose CTAs have started (a grid
    // starts only when every CTA of its predecessor has released it), so it ends without anything from this
    // grid: the thread polls the context's word for a bounded time, which costs less than waiting for the
    // whole preceding grid when several calls are in flight, and falls back to that wait.
    auto may_write = [&]() {
        if (need_seq <= 0) return;
        const volatile long long *done = reinterpret_cast<volatile long long *>(done_seq);
        // (the word learns of call s from the closing CTA of a later call; when the call needed is the one
        // directly before this one, that later call is this one, and only the wait below can tell)
        if (need_seq != LLONG_MAX && need_seq < my_seq - 1)
            for (int i = 0; i < 64 && *done < need_seq; ++i) __nanosleep(256);
        if (*done < need_seq) asm volatile("griddepcontrol.wait;" ::: "memory");
    };
    const int len = pp.off[n + 1] - pp.off[n];
    const int k = pp.cu_kv[n + 1] - pp.cu_kv[n];
    if (k == 0 || len == 0) {                                 // the same for every slice of the cluster
        if (closer && cu_kv && tid <= pp.n) {
            may_write();
            cu_kv[tid] = pp.cu_kv[tid];
        }
        close_call();
        return;
    }
    const int64_t T = pp.cu_kv[pp.n];

    // ---- 1. scores of this slice's tokens ----
    {
        // Every warp runs a pipeline of its own, without CTA-wide barriers: it takes the row groups
        // (32 rows, one per lane) w, w + 8, ... of the slice, copies a group's K rows of this head into its
        // private ring of n_stages buffers in column blocks of up to 8 chunks (128 bytes per row, chunks
        // XOR-swizzled by the row so that lane i walks row i without bank conflicts), and walks block
        // after block with the chain carried in a register.  n_stages - 1 blocks per warp are in flight
        // while one is walked; the conversion unit, the narrow pipe of this phase, is shared by all the
        // warps of the SM and stays busy because they drift apart.
        const int row_bytes = vpr * 16;
        const int per = (len + n_slices - 1) / n_slices;
        const int r0 = min(slice * per, len), r1 = min(r0 + per, len);
        const uint8_t *src = reinterpret_cast<const uint8_t *>(pp.k[n]) + (size_t)h * row_bytes;
        const size_t pitch = (size_t)hkv * row_bytes;          // bytes between consecutive tokens
        constexpr int kBlk = 8;                                // chunks per column block
        constexpr int kBufBytes = 32 * kBlk * 16;              // one buffer: 32 rows x 128 bytes
        const uint32_t wbase = (uint32_t)__cvta_generic_to_shared(stage) + warp * n_stages * kBufBytes;
        const uint8_t *wstage = stage + (size_t)warp * n_stages * kBufBytes;
        const int n_blk = (vpr + kBlk - 1) / kBlk;             // column blocks per row
        const int n_grp = (r1 - r0 + 31) / 32;                 // row groups of the slice
        const int my_grp = n_grp > warp ? (n_grp - warp + kSelThreads / 32 - 1) / (kSelThreads / 32) : 0;
        const int n_u = my_grp * n_blk;                        // (group, block) units of this warp, in order
        auto copy_unit = [&](int u) {                          // always commits a group, possibly empty
            if (u < n_u) {
                const int g = warp + (u / n_blk) * (kSelThreads / 32), blk = u % n_blk;
                const int c0 = r0 + g * 32, rows = min(32, r1 - c0);
                const int nc = min(kBlk, vpr - blk * kBlk);    // chunks of this block
                const uint32_t buf = wbase + (u % n_stages) * kBufBytes;
                for (int q = lane; q < rows * nc; q += 32) {
                    const int r = nc == kBlk ? q >> 3 : q / nc, ch = q - r * nc;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                                 ::"r"(buf + r * (kBlk * 16) + ((ch ^ (r & (kBlk - 1))) << 4)),
                                   "l"(src + (size_t)(c0 + r) * pitch + (blk * kBlk + ch) * 16) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        for (int u = 0; u < n_stages - 1; ++u) copy_unit(u);
        double sc = 0.0;
        for (int u = 0; u < n_u; ++u) {
            copy_unit(u + n_stages - 1);                       // into the buffer walked one unit ago
            if (n_stages == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
            else if (n_stages == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
            else asm volatile("cp.async.wait_group 3;" ::: "memory");
            __syncwarp();
            const int g = warp + (u / n_blk) * (kSelThreads / 32), blk = u % n_blk;
            const int row = r0 + g * 32 + lane;
            const int nc = min(kBlk, vpr - blk * kBlk);
            if (blk == 0) sc = 0.0;
            if (row < r1) {
                const uint4 *mine = reinterpret_cast<const uint4 *>(wstage + (size_t)(u % n_stages) * kBufBytes + lane * (kBlk * 16));
                const int sw = lane & (kBlk - 1);
                if (kDtype == FEDATTN_BF16) {
                    for (int v = 0; v < nc; ++v) {
                        const uint4 w = mine[v ^ sw];
                        sc = sq_acc_bf16x2(sc, w.x);
                        sc = sq_acc_bf16x2(sc, w.y);
                        sc = sq_acc_bf16x2(sc, w.z);
                        sc = sq_acc_bf16x2(sc, w.w);
                    }
                } else {
                    for (int v = 0; v < nc; ++v) {
                        const uint4 u4 = mine[v ^ sw];
                        const float x0 = __uint_as_float(u4.x), x1 = __uint_as_float(u4.y), x2 = __uint_as_float(u4.z),
                                    x3 = __uint_as_float(u4.w);
                        sc = __fma_rn((double)x0, (double)x0, sc);
                        sc = __fma_rn((double)x1, (double)x1, sc);
                        sc = __fma_rn((double)x2, (double)x2, sc);
                        sc = __fma_rn((double)x3, (double)x3, sc);
                    }
                }
                if (blk == n_blk - 1) keys[row] = (unsigned long long)__double_as_longlong(sc);
            }
            __syncwarp();                                      // the buffer is refilled n_stages - 1 units on
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");   // only empty groups are left
        // ---- 2. the other slices' keys ----
        cluster.sync();
        for (int q = 1; q < n_slices; ++q) {
            const int peer = (slice + q) % n_slices;
            const int p0 = min(peer * per, len), p1 = min(p0 + per, len);
            const unsigned long long *pk = cluster.map_shared_rank(keys, peer);
            for (int j = p0 + tid; j < p1; j += kSelThreads) keys[j] = pk[j];
        }
        // This CTA is done reading its peers; it may not exit before they are done reading it.  Arrive
        // now, wait at the very end: nothing after this touches distributed shared memory, and nobody
        // writes the keys a peer may still be reading.
        __syncthreads();                                      // the collected keys, for this CTA's own threads; also
                                                              // reconverges every warp for the aligned arrive
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }

    // ---- 3. selection ----
    // Bits that all keys share need no pass: (OR of all keys) ^ (AND of all keys) has a 1 exactly where
    // two keys differ.
    unsigned long long k_or = 0, k_and = ~0ULL;
    for (int j = tid; j < len; j += kSelThreads) {
        const unsigned long long key = keys[j];
        k_or |= key; k_and &= key;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        k_or |= __shfl_xor_sync(0xffffffffu, k_or, o);
        k_and &= __shfl_xor_sync(0xffffffffu, k_and, o);
    }
    if (lane == 0) { warp_or[warp] = k_or; warp_and[warp] = k_and; }
    __syncthreads();
    k_or = 0; k_and = ~0ULL;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) { k_or |= warp_or[w]; k_and &= warp_and[w]; }
    const unsigned long long diff = k_or ^ k_and, key0 = k_and;     // key0: the shared bits

    unsigned long long tau = key0;           // k-th largest score; k_rem rows equal to tau are kept
    int k_rem = k;
    if (diff != 0) {
        // first pass: the 8 bits that end at the highest differing bit, over all keys; the keys that fall
        // into the chosen bin are listed (my_rows doubles as the list) and later passes walk only the list
        int shift = max(63 - __clzll((long long)diff) - 7, 0);
        const unsigned long long above = shift + 8 >= 64 ? 0ULL : ~((1ULL << (shift + 8)) - 1ULL);
        unsigned long long prefix = key0 & above, mask = above;
        int n_cand = len;
        bool listed = false;
        for (;;) {
            const int nb = listed ? min(8, shift) : 8;
            if (listed) shift -= nb;
            hist[tid] = 0;
            if (tid == 0) sh_count = 0;
            __syncthreads();
            for (int i = tid; i < n_cand; i += kSelThreads) {
                const unsigned long long key = keys[listed ? my_rows[i] : i];
                if ((key & mask) == prefix) atomicAdd(&hist[(int)((key >> shift) & ((1u << nb) - 1u))], 1);
            }
            __syncthreads();
            // suffix sums over bins: S[b] = sum_{b' >= b} hist[b']
            const int mine = hist[tid];
            int incl = mine;   // inclusive suffix within warp: sum over lanes >= lane
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += up;
            }
            if (lane == 0) warp_tot[warp] = incl;
            __syncthreads();
            int above_w = 0;
#pragma unroll
            for (int w = 0; w < kSelThreads / 32; ++w)
                if (w > warp) above_w += warp_tot[w];
            const int S_b = incl + above_w;     // count of candidates with these bits >= tid
            const int S_next = S_b - mine;      // count with these bits > tid
            if (S_b >= k_rem && S_next < k_rem) {
                sh_bin = tid;
                sh_krem = k_rem - S_next;
            }
            __syncthreads();
            prefix |= (unsigned long long)sh_bin << shift;
            mask |= (unsigned long long)((1u << nb) - 1u) << shift;
            k_rem = sh_krem;
            if (shift == 0) break;
            if (!listed) {
                // list the keys of the chosen bin (order is irrelevant): one counter bump per warp
                for (int j0 = 0; j0 < len; j0 += kSelThreads) {
                    const int j = j0 + tid;
                    const bool in = j < len && (keys[j] & mask) == prefix;
                    const unsigned bal = __ballot_sync(0xffffffffu, in);
                    int base = 0;
                    if (lane == 0 && bal) base = atomicAdd(&sh_count, __popc(bal));
                    base = __shfl_sync(0xffffffffu, base, 0);
                    if (in) my_rows[base + __popc(bal & ((1u << lane) - 1u))] = (uint16_t)j;
                }
                __syncthreads();
                n_cand = sh_count;
                listed = true;
                if (n_cand <= kSelThreads) {
                    // Short list: thread i ranks candidate i against all others (broadcast reads, no more
                    // passes).  tau is the value v with #(> v) < k_rem <= #(>= v).
                    if (tid < n_cand) {
                        const unsigned long long mine_key = keys[my_rows[tid]];
                        int gt = 0, ge = 0;
                        for (int i = 0; i < n_cand; ++i) {
                            const unsigned long long other = keys[my_rows[i]];
                            gt += other > mine_key;
                            ge += other >= mine_key;
                        }
                        if (gt < k_rem && k_rem <= ge) { sh_tau = mine_key; sh_krem = k_rem - gt; }   // equal keys agree
                    }
                    __syncthreads();
                    prefix = sh_tau;
                    k_rem = sh_krem;
                    break;
                }
            }
        }
        tau = prefix;
    }
    __syncthreads();                                          // the list in my_rows is dead from here on

    // ordered compaction: thread tid owns indices [tid * per, (tid + 1) * per)
    const int per = (len + kSelThreads - 1) / kSelThreads;
    const int j_lo = min(tid * per, len), j_hi = min(j_lo + per, len);
    int n_gt = 0, n_eq = 0;
    for (int j = j_lo; j < j_hi; ++j) {
        const unsigned long long key = keys[j];
        n_gt += key > tau;
        n_eq += key == tau;
    }
    // exclusive block scan of (n_gt, n_eq), packed 16 + 16 bits (both <= 4096)
    unsigned packed = ((unsigned)n_gt << 16) | (unsigned)n_eq, incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    __syncthreads();                                          // warp_tot is free again
    if (lane == 31) warp_tot[warp] = (int)incl;
    __syncthreads();
    unsigned base = 0;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w)
        if (w < warp) base += (unsigned)warp_tot[w];
    const unsigned excl = base + incl - packed;
    int gt_before = (int)(excl >> 16), eq_before = (int)(excl & 0xffffu);
    // this CTA's share of the k outputs
    const int per_slice = (k + n_slices - 1) / n_slices;
    const int o_lo = min(slice * per_slice, k), o_hi = min(o_lo + per_slice, k);
    for (int j = j_lo; j < j_hi; ++j) {
        const unsigned long long key = keys[j];
        const bool gt = key > tau, eq = key == tau;
        if (gt || (eq && eq_before < k_rem)) {
            const int pos = gt_before + min(eq_before, k_rem);
            if (pos >= o_lo && pos < o_hi) my_rows[pos - o_lo] = (uint16_t)j;
        }
        gt_before += gt;
        eq_before += eq;
    }
    __syncthreads();

    // gather this slice: rows my_rows[0 .. o_hi - o_lo) of participant n, head h.  First write of this kernel.
    may_write();
    if (closer && cu_kv && tid <= pp.n) cu_kv[tid] = pp.cu_kv[tid];
    const int n_out = o_hi - o_lo;
    const int64_t out_row0 = (int64_t)h * T + pp.cu_kv[n] + o_lo;
    const uint4 *ksrc = reinterpret_cast<const uint4 *>(pp.k[n]), *vsrc = reinterpret_cast<const uint4 *>(pp.v[n]);
    // eight vectors of K and of V in flight per thread before the first store (a CTA gathers its rows in a few
    // round trips to memory: the gather is bound by that latency, not by bandwidth)
    constexpr int kGatherUnroll = 8;
    for (int i0 = tid; i0 < n_out * vpr; i0 += kSelThreads * kGatherUnroll) {
        uint4 kk[kGatherUnroll], vv[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int i = i0 + u * kSelThreads;
            if (i < n_out * vpr) {
                const int r = i / vpr, vi = i - r * vpr;
                const int64_t src = ((int64_t)my_rows[r] * hkv + h) * vpr + vi;
                kk[u] = ld_stream(ksrc + src);
                vv[u] = ld_stream(vsrc + src);
            }
        }
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int i = i0 + u * kSelThreads;
            if (i < n_out * vpr) {
                const int r = i / vpr, vi = i - r * vpr;
                const int64_t dst = (out_row0 + r) * vpr + vi;
                k_agg[dst] = kk[u];
                v_agg[dst] = vv[u];
            }
        }
    }
    for (int r = tid; r < n_out; r += kSelThreads) {
        if (kv_pos) kv_pos[out_row0 + r] = pp.off[n] + my_rows[r];
        if (sel_idx_out) sel_idx_out[out_row0 + r] = my_rows[r];
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    close_call();
}

cudaError_t launch_topk_fused(const PartsParams &pp, int hkv, int d, int dtype, void *k_agg, void *v_agg,
                              int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out, Context *ctx, cudaStream_t s)
{
    const int device = ctx->device, sm_count = ctx->sm_count;
    int64_t *launches = &ctx->launches;
    if (pp.cu_kv[pp.n] == 0 && !cu_kv) return cudaSuccess;
    const int elt = dtype == FEDATTN_BF16 ? 2 : 4;
    int early;
    long long *done_seq = reinterpret_cast<long long *>(ctx->workspace + kDoneSeqOffset);
    long long my_seq = 0;
    int64_t need_seq = 0;
    {
        const size_t row_bytes = (size_t)hkv * d * elt;
        const size_t T = (size_t)pp.cu_kv[pp.n];
        MemRange in[2 * kMaxP];
        for (int i = 0; i < pp.n; ++i) {
            const size_t bytes = (size_t)(pp.off[i + 1] - pp.off[i]) * row_bytes;
            in[2 * i] = {pp.k[i], bytes};
            in[2 * i + 1] = {pp.v[i], bytes};
        }
        const MemRange out[5] = {{k_agg, T * row_bytes}, {v_agg, T * row_bytes}, {kv_pos, kv_pos ? T * hkv * 4 : 0},
                                 {cu_kv, cu_kv ? (size_t)(pp.n + 1) * 4 : 0}, {sel_idx_out, sel_idx_out ? T * hkv * 4 : 0}};
        const EarlyStart es = early_start(device, s, in, 2 * pp.n, out, 5, true, done_seq, &ctx->agg_seq, &ctx->agg_key);
        early = es.early ? 1 : 0;
        my_seq = es.seq;
        need_seq = es.need_seq;
    }
    const int vpr = d * elt / 16;
    int max_len = 0;
    for (int i = 0; i < pp.n; ++i) max_len = max(max_len, pp.off[i + 1] - pp.off[i]);
    if (max_len > kSelMaxLen) return cudaErrorInvalidValue;
    // Shared memory per CTA: keys (8 B) and kept rows (2 B) per token of the longest participant, then
    // the staging buffers.  As many buffers (2..4) as still let kCtasPerSm CTAs share an SM: what is in
    // flight from HBM is all but one of them.  More resident CTAs matter more than deeper rings: CTAs in
    // different phases (scores, selection, gather), also of consecutive calls, keep HBM busy.
    const int stage_bytes = (kSelThreads / 32) * 32 * 128;    // one buffer per warp: 32 rows x 128 bytes
    const int fixed = (max_len * 10 + 15) & ~15;
    const int per_cta = (228 * 1024) / kCtasPerSm - 1024 /*reserved per CTA*/ - 2048 /*static*/;
    int n_stages = (per_cta - fixed) / stage_bytes;
    n_stages = n_stages < 2 ? 2 : (n_stages > 4 ? 4 : n_stages);
    const int smem = fixed + n_stages * stage_bytes;
    static bool attr_set[64] = {};                            // the attribute is per device
    if (!attr_set[device & 63]) {
        const int most = 227 * 1024 - 2048;
        cudaError_t e = cudaFuncSetAttribute(topk_fused_kernel<FEDATTN_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(topk_fused_kernel<FEDATTN_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
        if (e != cudaSuccess) return e;
        attr_set[device & 63] = true;
    }
    // slices per (head, participant): a power of two <= 8 (one cluster), about two CTAs per SM in total, and
    // every slice keeps at least one token per lane of the CTA (a lane walks one key row at a time)
    const int pairs = hkv * pp.n;
    int slices = 1;
    while (slices * 2 <= kMaxSlices && pairs * slices * 2 <= sm_count && max_len >= kSelThreads * slices * 2) slices *= 2;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(hkv, pp.n, slices);
    cfg.blockDim = dim3(kSelThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = slices;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = dtype == FEDATTN_BF16
                        ? cudaLaunchKernelEx(&cfg, topk_fused_kernel<FEDATTN_BF16>, pp, hkv, vpr, n_stages, max_len, early, my_seq,
                                             (long long)need_seq, done_seq, (uint4 *)k_agg, (uint4 *)v_agg, kv_pos, cu_kv, sel_idx_out)
                        : cudaLaunchKernelEx(&cfg, topk_fused_kernel<FEDATTN_F32>, pp, hkv, vpr, n_stages, max_len, early, my_seq,
                                             (long long)need_seq, done_seq, (uint4 *)k_agg, (uint4 *)v_agg, kv_pos, cu_kv, sel_idx_out);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- indexed gather ------------------------------------------------------------------------------
// One 16-byte vector per thread and step, kGatherBatch steps in flight.  Launched with programmatic stream
// serialization like the fused kernel above: indices and rows are read at once (unless they might be
// outputs of a grid that is still running: early == 0), everything is written after griddepcontrol.wait.
constexpr int kGatherBatch = 4;

__global__ void __launch_bounds__(256)
gather_kernel(const PartsParams pp, int hkv, int64_t vpr /* 16-byte vectors per (row, head) */,
              const int32_t *sel_idx, uint4 *k_agg, uint4 *v_agg, int32_t *kv_pos, int32_t *cu_kv,
              int32_t *sel_idx_out, int32_t *status, int early)
{
    if (!early) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited = !early;
    const int64_t T = pp.cu_kv[pp.n];
    const int64_t total = (int64_t)hkv * T * vpr;
    const bool is_v = blockIdx.y != 0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i0 = tid; i0 < total; i0 += stride * kGatherBatch) {
        uint4 val[kGatherBatch];
        int32_t idx[kGatherBatch], pos[kGatherBatch];
        bool keep[kGatherBatch], first[kGatherBatch];
        bool bad = false;
#pragma unroll
        for (int b = 0; b < kGatherBatch; ++b) {
            const int64_t i = i0 + b * stride;
            keep[b] = false; first[b] = false; idx[b] = 0; pos[b] = 0;
            if (i >= total) continue;
            const int64_t rowid = i / vpr;               // h * T + t
            const int vi = (int)(i - rowid * vpr);
            const int h = (int)(rowid / T);
            const int32_t t = (int32_t)(rowid - (int64_t)h * T);
            const int n = find_segment(pp.cu_kv, pp.n, t);
            const int32_t j = __ldg(sel_idx + rowid);
            const int32_t len = pp.off[n + 1] - pp.off[n];
            // in range, and strictly above its predecessor inside the same (head, participant) block: the
            // aggregate's positions must come out ascending, which the attention over it relies on
            if (j < 0 || j >= len || (t > pp.cu_kv[n] && __ldg(sel_idx + rowid - 1) >= j)) {
                bad |= vi == 0;
                if (j < 0 || j >= len) continue;
            }
            const uint4 *src = reinterpret_cast<const uint4 *>(is_v ? pp.v[n] : pp.k[n]) +
                               ((int64_t)j * hkv + h) * vpr + vi;
            val[b] = ld_stream(src);
            keep[b] = true; first[b] = vi == 0; idx[b] = j; pos[b] = pp.off[n] + j;
        }
        if (!waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        if (bad) atomicMax(status, (int32_t)FEDATTN_ERR_INDEX);
#pragma unroll
        for (int b = 0; b < kGatherBatch; ++b) {
            if (!keep[b]) continue;
            const int64_t i = i0 + b * stride;
            (is_v ? v_agg : k_agg)[i] = val[b];
            if (first[b] && !is_v) {
                const int64_t rowid = i / vpr;
                if (kv_pos) kv_pos[rowid] = pos[b];
                if (sel_idx_out && sel_idx_out != sel_idx) sel_idx_out[rowid] = idx[b];
            }
        }
    }
    if (!is_v && cu_kv && tid <= pp.n) {
        if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
        cu_kv[tid] = pp.cu_kv[tid];
    }
}

cudaError_t launch_gather(const PartsParams &pp, int hkv, int d, int elt_bytes, const int32_t *sel_idx,
                          void *k_agg, void *v_agg, int32_t *kv_pos, int32_t *cu_kv, int32_t *sel_idx_out,
                          int32_t *status, int device, int sm_count, cudaStream_t s, int64_t *launches)
{
    const int64_t vpr = (int64_t)d * elt_bytes / 16;
    const int64_t T = pp.cu_kv[pp.n];
    const int64_t total = (int64_t)hkv * T * vpr;
    // the whole grid is resident at once (the next grid of the stream starts when every CTA of this one has)
    int64_t blocks = (total + 256 * kGatherBatch - 1) / (256 * kGatherBatch);
    if (blocks > (int64_t)sm_count * 3) blocks = (int64_t)sm_count * 3;
    if (blocks < 1) blocks = 1;
    int early;
    {
        const size_t row_bytes = (size_t)hkv * d * elt_bytes;
        MemRange in[2 * kMaxP + 1];
        for (int i = 0; i < pp.n; ++i) {
            const size_t bytes = (size_t)(pp.off[i + 1] - pp.off[i]) * row_bytes;
            in[2 * i] = {pp.k[i], bytes};
            in[2 * i + 1] = {pp.v[i], bytes};
        }
        in[2 * pp.n] = {sel_idx, (size_t)T * hkv * 4};
        const MemRange out[5] = {{k_agg, (size_t)T * row_bytes}, {v_agg, (size_t)T * row_bytes}, {kv_pos, kv_pos ? (size_t)T * hkv * 4 : 0},
                                 {cu_kv, cu_kv ? (size_t)(pp.n + 1) * 4 : 0},
                                 {sel_idx_out, (sel_idx_out && sel_idx_out != sel_idx) ? (size_t)T * hkv * 4 : 0}};
        early = early_start(device, s, in, 2 * pp.n + 1, out, 5).early ? 1 : 0;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)blocks, 2, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, gather_kernel, pp, hkv, vpr, sel_idx, (uint4 *)k_agg, (uint4 *)v_agg, kv_pos, cu_kv,
                                             sel_idx_out, status, early);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace fedattn
