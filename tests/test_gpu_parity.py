"""GPU parity: the CUDA path, called through the C-ABI binding, against the fp64 CPU oracle on the
same seeded inputs.  Bars: bit-exact for offsets / positions / selected indices / copied bytes;
max-abs 1e-4 for fp32 inputs; max-abs 2e-2 for bf16 inputs with O(1) outputs."""
import numpy as np
import pytest
import torch

import fedattn_inputs as fi
from helpers import LSE_TOL, TOL, Runner, check_close, dev, fa, host

pytestmark = pytest.mark.gpu


def split(x, lens):
    return np.split(x, np.cumsum(lens)[:-1])


def gen(seed, lens, hq, hkv, d, dtype, gain=1.0):
    w = fi.Workload("t", seed, tuple(int(x) for x in lens), hq, hkv, d, dtype, gain)
    return w.qkv()


def test_buffers_on_16_byte_boundaries_and_ragged_tiles(oracle):
    """Q, K, V and O at addresses that are multiples of 16 but not of 32 bytes, with full and ragged
    128-row tiles in one call: rows leave through both store paths (whole warps of rows in bulk, the
    rows of a ragged warp one by one) and both must land where the layout says."""
    lens = [256, 130, 300, 128, 17]
    hq, hkv, d = 8, 2, 128
    q, k, v = gen(91, lens, hq, hkv, d, "bf16")
    L = sum(lens)
    m = fa()
    shape = m.Shape(len(lens), hq, hkv, d, m.BF16, 1, 0.0)
    ctx = m.Context(shape, L, L)

    def shifted(x):                       # the same values, 16 bytes further
        flat = torch.empty(x.numel() + 8, dtype=torch.bfloat16, device="cuda")
        view = flat[8:].view(x.shape)
        view.copy_(x)
        assert view.data_ptr() % 32 == 16
        return view

    qd, kd, vd = (shifted(dev(x, "bf16")) for x in (q, k, v))
    o = shifted(torch.full_like(dev(q, "bf16"), float("nan")))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    m.fedattn_local(ctx, shape, qd, kd, vd, cu, o)
    assert ctx.poll() == 0
    oo, _ = oracle.local(q, k, v, lens)
    check_close(host(o), oo, TOL["bf16"], "local, shifted buffers")
    o2 = shifted(torch.full_like(dev(q, "bf16"), float("nan")))
    m.fedattn_sync(ctx, shape, qd, None, kd, vd, None, L, False, o2)
    assert ctx.poll() == 0
    oo, _ = oracle.sync(q, k, v)
    check_close(host(o2), oo, TOL["bf16"], "sync, shifted buffers")
    assert ctx.tensor_core_launch_count() == 2


# ---------------------------------------------------------------------------------------------
# config 1: fp32, N=2 x 128, 4 heads, d=64 -- full comparison, local and sync
# ---------------------------------------------------------------------------------------------
def test_cfg1_fp32_local_and_sync(oracle):
    w = fi.cfg1()
    q, k, v = w.qkv()
    r = Runner(2, 4, 4, 64, "f32", 256)
    o, lse = r.local(q, k, v, w.seqlens)
    oo, ol = oracle.local(q, k, v, w.seqlens)
    e1 = check_close(o, oo, TOL["f32"], "cfg1 local o")
    check_close(lse, ol, TOL["f32"], "cfg1 local lse")
    agg = r.aggregate(fa().AGG_CONCAT, split(k, w.seqlens), split(v, w.seqlens))
    ka, va, pos, cu = oracle.aggregate_concat(split(k, w.seqlens), split(v, w.seqlens))
    assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
    o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"])
    oo, ol = oracle.sync(q, ka, va, kv_pos=pos)
    check_close(o, oo, TOL["f32"], "cfg1 sync o")
    check_close(lse, ol, TOL["f32"], "cfg1 sync lse")
    assert np.abs(oo).max() > 0.1 and e1 < TOL["f32"]


@pytest.mark.parametrize("dtype,hq,hkv,d", [("f32", 4, 2, 32), ("f32", 2, 2, 128), ("bf16", 4, 2, 64),
                                            ("bf16", 8, 2, 128), ("bf16", 4, 4, 128), ("bf16", 6, 2, 128)])
@pytest.mark.parametrize("causal", [True, False])
def test_ragged_segments_local_and_sync(oracle, dtype, hq, hkv, d, causal):
    """Ragged lengths incl. 1, 0 and non-multiples of the 128-row tile; several tiles per segment."""
    lens = [1, 130, 0, 257, 64, 300]
    q, k, v = gen(11, lens, hq, hkv, d, dtype)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens), causal=causal)
    o, lse = r.local(q, k, v, lens)
    oo, ol = oracle.local(q, k, v, lens, causal=causal)
    check_close(o, oo, TOL[dtype], "local o")
    check_close(lse, ol, LSE_TOL[dtype], "local lse")
    o, lse = r.sync(q, k, v)
    oo, ol = oracle.sync(q, k, v, causal=causal)
    check_close(o, oo, TOL[dtype], "sync o")
    check_close(lse, ol, LSE_TOL[dtype], "sync lse")
    # twice the same call: bitwise identical
    o2, _ = r.sync(q, k, v)
    assert np.array_equal(o, o2)


def test_single_participant_and_tiny(oracle):
    for lens, hq, hkv in [([1], 4, 4), ([5], 8, 2), ([129], 4, 1), ([128, 128], 4, 2), ([127, 1, 128], 4, 2)]:
        q, k, v = gen(5, lens, hq, hkv, 128, "bf16")
        r = Runner(len(lens), hq, hkv, 128, "bf16", sum(lens))
        check_close(r.local(q, k, v, lens)[0], oracle.local(q, k, v, lens)[0], TOL["bf16"], str(lens))
        check_close(r.sync(q, k, v)[0], oracle.sync(q, k, v)[0], TOL["bf16"], str(lens))


def test_growing_logits_exercise_the_rescale_path(oracle):
    """Logits that grow along the key axis force the running-maximum reference to move many times
    (within a tile and across tiles), so O, P and l are rescaled on the way."""
    lens = [300, 260]
    q, k, v = gen(13, lens, 4, 2, 128, "bf16")
    ramp = (np.arange(sum(lens), dtype=np.float32) % 300 / 6.0)[:, None, None]
    q = fi.round_to_bf16(np.abs(q))
    k = fi.round_to_bf16(np.abs(k) * ramp)           # logits ~ +ramp * O(10): far beyond 2^8 per chunk
    r = Runner(2, 4, 2, 128, "bf16", sum(lens))
    o, lse = r.local(q, k, v, lens)
    oo, ol = oracle.local(q, k, v, lens)
    check_close(o, oo, TOL["bf16"], "rescale local")
    assert np.abs(lse - ol).max() / np.abs(ol).max() < 1e-3
    o, _ = r.sync(q, k, v)
    check_close(o, oracle.sync(q, k, v)[0], TOL["bf16"], "rescale sync")
    # and the opposite: the first keys dominate, later chunks underflow
    k2 = fi.round_to_bf16(np.abs(k[::-1].copy()))
    check_close(r.sync(q, k2, v)[0], oracle.sync(q, k2, v)[0], TOL["bf16"], "falling logits")


def test_sync_with_explicit_query_positions(oracle):
    """One participant's rows against the global KV, positions given explicitly."""
    lens = [100, 60, 140]
    q, k, v = gen(6, lens, 4, 2, 128, "bf16")
    r = Runner(3, 4, 2, 128, "bf16", 300)
    qp = np.arange(100, 160, dtype=np.int32)
    tc0 = r.ctx.tensor_core_launch_count()
    o, lse = r.sync(q[100:160], k, v, q_pos=qp)
    assert r.ctx.tensor_core_launch_count() == tc0 + 1          # explicit positions stay on the tensor-core kernel
    oo, ol = oracle.sync(q[100:160], k, v, q_pos=qp)
    check_close(o, oo, TOL["bf16"], "q_pos")
    check_close(lse, ol, LSE_TOL["bf16"], "q_pos lse")
    check_close(o, oracle.sync(q, k, v)[0][100:160], TOL["bf16"], "q_pos vs packed")


@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("f32", 4, 2, 64)])
@pytest.mark.parametrize("kind,lens", [("interleaved", [300, 300, 300]), ("interleaved", [130, 1, 517, 64]),
                                       ("random", [257, 400, 90])])
def test_general_index_sets_through_explicit_positions(oracle, dtype, hq, hkv, d, kind, lens):
    """Participants that hold general ordered index sets of the global sequence (Sec. IV-A), e.g.
    token t at participant t mod N: the aggregate concatenated in participant order has key positions
    that go up and down, and the queries carry their positions explicitly.  Every (query, key) pair
    is tested on its own positions; the result equals the oracle's sync attention."""
    sets = fi.index_sets(17, lens, kind)
    pos = np.concatenate(sets).astype(np.int32)
    assert np.any(np.diff(pos) < 0)
    q, k, v = gen(81, lens, hq, hkv, d, dtype)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens))
    tc0 = r.ctx.tensor_core_launch_count()
    o, lse = r.sync(q, k, v, kv_pos=pos, q_pos=pos)
    if dtype == "bf16":
        assert r.ctx.tensor_core_launch_count() == tc0 + 1
    oo, ol = oracle.sync(q, k, v, kv_pos=pos, q_pos=pos)
    check_close(o, oo, TOL[dtype], "index sets %s" % kind)
    check_close(lse, ol, LSE_TOL[dtype], "index sets %s lse" % kind)
    # one participant's rows alone, head-major aggregate (per-head position arrays)
    n = len(lens) - 1
    r0 = sum(lens[:n])
    kh = np.ascontiguousarray(np.transpose(k, (1, 0, 2))); vh = np.ascontiguousarray(np.transpose(v, (1, 0, 2)))
    posh = np.ascontiguousarray(np.tile(pos, (hkv, 1)))
    o, lse = r.sync(q[r0:], kh, vh, kv_pos=posh, q_pos=pos[r0:], head_major=True)
    check_close(o, oo[r0:], TOL[dtype], "index sets %s, one participant" % kind)
    check_close(lse, ol[r0:], LSE_TOL[dtype], "index sets %s, one participant lse" % kind)


def test_unsorted_key_positions_without_query_positions_raise_a_status(oracle):
    """The prefix-count mask of the bf16 head_dim 128 kernel needs non-decreasing kv_pos.  Positions
    that go down are reported (status 7), not silently mis-masked; the same input with explicit
    query positions is handled exactly."""
    lens = [200, 200]
    pos = np.concatenate(fi.index_sets(3, lens, "interleaved")).astype(np.int32)
    q, k, v = gen(82, lens, 4, 2, 128, "bf16")
    r = Runner(2, 4, 2, 128, "bf16", 400)
    m = fa()
    qd, kd, vd = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    pd = torch.from_numpy(pos).cuda()
    o = torch.zeros_like(qd)
    m.fedattn_sync(r.ctx, r.shape, qd, None, kd, vd, pd, 400, False, o)
    assert r.poll() == 7
    qp = np.arange(400, dtype=np.int32)
    o, _ = r.sync(q, k, v, kv_pos=pos, q_pos=qp)
    check_close(o, oracle.sync(q, k, v, kv_pos=pos, q_pos=qp)[0], TOL["bf16"], "unsorted kv_pos with q_pos")
    sorted_pos = np.sort(pos)
    sp = torch.from_numpy(sorted_pos).cuda()
    m.fedattn_sync(r.ctx, r.shape, qd, None, kd, vd, sp, 400, False, torch.zeros_like(qd))
    assert r.poll() == 0                                         # non-decreasing positions pass the check


# ---------------------------------------------------------------------------------------------
# aggregation
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_concat_is_bit_exact(oracle, dtype):
    lens = [3, 0, 257, 1, 1000]
    _, k, v = gen(7, lens, 2, 2, 64, dtype)
    r = Runner(len(lens), 2, 2, 64, dtype, sum(lens))
    agg = r.aggregate(fa().AGG_CONCAT, split(k, lens), split(v, lens))
    ka, va, pos, cu = oracle.aggregate_concat(split(k, lens), split(v, lens))
    assert agg["status"] == 0
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
    assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_topk_indices_bit_exact_with_ties(oracle, dtype):
    lens = [300, 1, 64, 1000, 7]
    ksel = [75, 1, 0, 250, 7]
    hkv, d = 4, 128
    _, k, v = gen(8, lens, hkv, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    kp[0][17] = kp[0][3]; kp[0][200] = kp[0][3]; kp[0][40, 1] = -kp[0][41, 1]     # planted ties
    kp[3][:] = kp[3][0]                                                           # all equal => first k
    r = Runner(len(lens), hkv, hkv, d, dtype, sum(lens))
    agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    assert agg["status"] == 0
    assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
    assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
    assert list(sel[0, cu[3]:cu[4]]) == list(range(250))


def test_topk_max_length_many_slices_and_degenerate_scores(oracle):
    """Longest supported segment (4096), slices of one (head, participant) spread over a cluster,
    k = 1 / k = L_n, near-constant scores (selection decided in the lowest bits) and long runs of
    exactly equal scores (tie rule over many candidates)."""
    lens = [4096, 513]
    hkv, d = 2, 128
    _, k, v = gen(21, lens, hkv, hkv, d, "bf16")
    kp, vp = split(k, lens), split(v, lens)
    kp[0][1000:3000] = kp[0][1000]                    # 2000 equal scores in the middle
    kp[1][:, 1, :] = 1.0                              # head 1 of participant 1: all scores equal
    kp[1][7, 1, 0] = 1.0078125                        # ... except one, larger by one bf16 step
    r = Runner(len(lens), hkv, hkv, d, "bf16", sum(lens))
    for ksel in ([1024, 128], [1, 513], [4096, 1], [2500, 0]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert agg["status"] == 0
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel), ksel
        assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)


@pytest.mark.parametrize("d", [128, 64, 40])
def test_topk_zero_and_subnormal_terms(oracle, d):
    """Rows with exact zeros, bf16 subnormals and all-zero rows (padding): their scores must still be
    the exact chain, also where rows differ only by such terms (scores of the order of 1e-80)."""
    lens = [300, 97]
    hkv = 2
    _, k, v = gen(23, lens, hkv, hkv, d, "bf16")
    rng = np.random.default_rng(23)
    k[rng.random(k.shape) < 0.05] = 0.0                               # scattered zeros, any column
    tiny = np.float32(2.0 ** -130)                                    # a bf16 subnormal
    k[10:40] = 0.0                                                    # all-zero rows
    k[20:30, :, d - 1] = tiny * np.arange(1, 11, dtype=np.float32)[:, None]   # ... some with one subnormal term
    k[40:50, :, ::2] = tiny                                           # rows of zeros and subnormals only
    k[305:320, :, d // 2:] = 0.0                                      # half-zero rows in the second participant
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hkv, hkv, d, "bf16", sum(lens))
    for ksel in ([280, 50], [295, 97], [5, 1]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert agg["status"] == 0
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel), ksel
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)


@pytest.mark.parametrize("d", [128, 64])
def test_topk_scores_around_the_exactness_bound(oracle, d):
    """The bf16 score kernel sums a row in tree order when it can prove that no addition of the defined
    chain rounds (row sum below 2^53 times the smallest term's unit), and walks the chain otherwise.
    Rows built around that bound: groups of rows that share their large elements and differ only in a
    tiny element (exponents on both sides of the bound, full and minimal mantissa) and in where it
    sits in the row, so that inside a group the order is decided by the last bits of the score."""
    rng = np.random.default_rng(31)
    hkv, groups, per_group = 2, 90, 8
    L = groups * per_group
    base = fi.round_to_bf16(rng.standard_normal((groups, 1, hkv, d)).astype(np.float32) * np.float32(2.0))
    k = np.repeat(base, per_group, axis=1).reshape(L, hkv, d).copy()
    tiny_exp = [-18, -17, -16, -15, -14, -13]                        # the bound sits near 2^-16 .. 2^-15 for sums of a few hundred
    for g in range(groups):
        for j in range(per_group):
            row = g * per_group + j
            e = tiny_exp[(g + j) % len(tiny_exp)]
            mant = np.float32(1.9921875) if (g // 2 + j) % 2 else np.float32(1.0)     # 8-bit mantissa 0xff or 0x80
            col = [0, d // 2, d - 1, 3][j % 4]
            k[row, :, col] = mant * np.float32(2.0) ** e * (1 if j % 2 else -1)
    k = fi.round_to_bf16(k)
    v = fi.round_to_bf16(rng.standard_normal((L, hkv, d)).astype(np.float32))
    kp, vp = [k[:L // 2], k[L // 2:]], [v[:L // 2], v[L // 2:]]
    r = Runner(2, hkv, hkv, d, "bf16", L)
    for ksel in ([L // 4, L // 4], [101, 257], [7, 355], [L // 2 - 3, 1]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert agg["status"] == 0
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel), ksel
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)


@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("bf16", 32, 8, 128), ("f32", 4, 2, 64)])
def test_token_level_selection_and_sync_over_it(oracle, dtype, hq, hkv, d):
    """Token-level selection: one score per token over all KV heads (a chain of Hkv * d terms), indices
    bit-exact; the token-major sparse KV then feeds the sync attention with a shared kv_pos."""
    lens = [300, 97, 513]
    q, k, v = gen(24, lens, hq, hkv, d, dtype)
    k[310:330] = k[305]                                               # equal scores across tokens
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens))
    for ksel in ([75, 24, 128], [300, 0, 1], [0, 0, 0]):
        agg = r.aggregate(fa().AGG_TOPK_TOKEN, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk_token(kp, vp, ksel)
        assert agg["status"] == 0
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel), ksel
        assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
        o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"], head_major=False)
        oo, ol = oracle.sync(q, ka, va, kv_pos=pos)
        check_close(o, oo, TOL[dtype], "sync over token-level selection %s" % ksel)
        check_close(lse, ol, LSE_TOL[dtype], "sync over token-level selection lse %s" % ksel)


def test_topk_fp32_head_dim_128(oracle):
    lens = [700, 300]
    hkv, d = 8, 128
    _, k, v = gen(22, lens, hkv, hkv, d, "f32")
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hkv, hkv, d, "f32", sum(lens))
    ksel = [175, 75]
    agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)



def test_indexed_aggregation_and_bad_index_status(oracle):
    lens = [50, 20, 30]
    ksel = [5, 0, 30]
    hkv, d = 2, 64
    _, k, v = gen(9, lens, hkv, hkv, d, "bf16")
    kp, vp = split(k, lens), split(v, lens)
    rng = np.random.default_rng(0)
    sel = np.stack([np.concatenate([np.sort(rng.choice(50, 5, replace=False)), np.arange(30)]) for _ in range(hkv)])
    r = Runner(3, hkv, hkv, d, "bf16", 100)
    agg = r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)
    ka, va, pos, cu = oracle.aggregate_indexed(kp, vp, ksel, sel)
    assert agg["status"] == 0
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
    assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
    bad = sel.copy()
    bad[1, 2] = 50                                   # out of range for participant 0 (L_0 = 50)
    agg = r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=bad)
    assert agg["status"] == 6                        # reported, not faulted; context still usable
    assert r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)["status"] == 0
    unsorted = sel.copy()
    unsorted[0, 1], unsorted[0, 2] = sel[0, 2], sel[0, 1]      # in range, but not ascending inside participant 0's block
    assert r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=unsorted)["status"] == 6
    dup = sel.copy()
    dup[1, 6] = dup[1, 5]                            # a repeated index is not ascending either
    assert r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=dup)["status"] == 6
    assert r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)["status"] == 0


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_sparse_sync_small_incl_empty_rows_and_excluded_participant(oracle, dtype):
    lens = [140, 90, 260]
    hq, hkv, d = 8, 2, 128
    q, k, v = gen(10, lens, hq, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(3, hq, hkv, d, dtype, sum(lens))
    for ksel in ([35, 23, 65], [0, 30, 100], [140, 90, 260], [0, 0, 0]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
        o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"], head_major=True)
        oo, ol = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True)
        check_close(o, oo, TOL[dtype], "sparse sync %s" % ksel)
        check_close(lse, ol, LSE_TOL[dtype], "sparse sync lse %s" % ksel)
    # rows of the first participant see nothing when it is excluded: zeros and -inf
    assert np.all(o[:140] == 0)


# ---------------------------------------------------------------------------------------------
# sync block with sparse KV exchange: own segment complete + sparsified remote keys
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("f32", 4, 2, 64)])
def test_sync_exchange_small(oracle, dtype, hq, hkv, d):
    lens = [140, 90, 260, 33]
    q, k, v = gen(41, lens, hq, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens))
    for ksel in ([35, 23, 65, 8], [140, 90, 260, 33], [0, 0, 0, 0], [0, 90, 0, 5]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
        o, lse = r.sync_exchange(q, k, v, lens, agg)
        oo, ol = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
        check_close(o, oo, TOL[dtype], "sync exchange %s" % ksel)
        check_close(lse, ol, LSE_TOL[dtype], "sync exchange lse %s" % ksel)


@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("f32", 4, 2, 64)])
@pytest.mark.parametrize("causal", [True, False])
def test_sync_exchange_with_a_seeded_random_selection(oracle, dtype, hq, hkv, d, causal):
    """The sparsity-ratio experiment samples the exchanged rows at random (Sec. VI).  The draw is an
    input: seeded indices per (participant, KV head) -> indexed aggregation -> local attention +
    remote-only sync + merge, against the oracle's exchange block on the same draw; causal and
    bidirectional (Sec. III-B)."""
    lens = [140, 90, 260, 33, 129]
    q, k, v = gen(43, lens, hq, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens), causal=causal)
    for num, den in ((1, 4), (1, 2), (1, 1), (0, 1)):
        ksel = [(n * num + den - 1) // den for n in lens]
        sel = fi.random_selection(7, lens, ksel, hkv)
        agg = r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)
        ka, va, pos, cu = oracle.aggregate_indexed(kp, vp, ksel, sel)
        assert agg["status"] == 0
        assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
        o, lse = r.sync_exchange(q, k, v, lens, agg)
        oo, ol = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu, causal=causal)
        check_close(o, oo, TOL[dtype], "random exchange %d/%d causal=%s" % (num, den, causal))
        check_close(lse, ol, LSE_TOL[dtype], "random exchange lse %d/%d causal=%s" % (num, den, causal))


@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("bf16", 6, 2, 128), ("f32", 4, 2, 64)])
def test_sync_exchange_bidirectional(oracle, dtype, hq, hkv, d):
    """causal = 0: own segment complete (all of it) + every exchanged key of the other participants.
    The remote keys of a participant are two ranges of the aggregate (before and after its own
    rows); segments whose boundaries fall inside a 128-key tile, an excluded participant, top-k and
    full exchange."""
    lens = [140, 90, 260, 33, 385]
    q, k, v = gen(44, lens, hq, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens), causal=False)
    for ksel in ([35, 23, 65, 8, 100], [140, 90, 260, 33, 385], [0, 0, 0, 0, 0], [128, 0, 128, 0, 1], [0, 90, 0, 0, 0]):
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
        o, lse = r.sync_exchange(q, k, v, lens, agg)
        oo, ol = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu, causal=False)
        check_close(o, oo, TOL[dtype], "bidirectional exchange %s" % ksel)
        check_close(lse, ol, LSE_TOL[dtype], "bidirectional exchange lse %s" % ksel)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_merge_of_partial_results_closed_form_and_empty_parts(dtype):
    """fedattn_merge against the closed form (softmax over a disjoint union of key sets): weights
    exp(lse - max) normalised; a part with lse = -inf carries no weight; two empty parts give 0, -inf."""
    rng = np.random.default_rng(9)
    L, hq, d = 70, 4, 128 if dtype == "bf16" else 64
    o_a = fi.round_to_bf16(rng.standard_normal((L, hq, d)).astype(np.float32)) if dtype == "bf16" else rng.standard_normal((L, hq, d)).astype(np.float32)
    o_b = fi.round_to_bf16(rng.standard_normal((L, hq, d)).astype(np.float32)) if dtype == "bf16" else rng.standard_normal((L, hq, d)).astype(np.float32)
    lse_a = (rng.standard_normal((L, hq)) * 30).astype(np.float32)
    lse_b = (rng.standard_normal((L, hq)) * 30).astype(np.float32)
    lse_a[3] = -np.inf; o_a[3] = 0                    # empty first part
    lse_b[5] = -np.inf; o_b[5] = 0                    # empty second part
    lse_a[7] = lse_b[7] = -np.inf; o_a[7] = o_b[7] = 0    # both empty
    lse_b[9] = lse_a[9]                               # equal weights: the mean
    r = Runner(2, hq, hq, d, dtype, L)
    o, lse = r.merge(o_a.astype(np.float64), lse_a, o_b.astype(np.float64), lse_b)
    la, lb = lse_a.astype(np.float64), lse_b.astype(np.float64)
    m = np.maximum(la, lb); m = np.where(np.isfinite(m), m, 0.0)
    wa, wb = np.exp(la - m), np.exp(lb - m)
    z = wa + wb
    want = (o_a * wa[..., None] + o_b * wb[..., None]) / np.where(z > 0, z, 1.0)[..., None]
    with np.errstate(divide="ignore"):
        want_lse = m + np.log(z)
    check_close(o, want, TOL[dtype], "merge o")
    check_close(lse, want_lse, 1e-4 * 30, "merge lse")
    assert np.all(o[7] == 0) and np.all(np.isneginf(lse[7]))
    check_close(o[9], 0.5 * (o_a[9].astype(np.float64) + o_b[9]), TOL[dtype], "merge, equal weights")


def test_cfg4_sync_exchange_full_size_sampled(oracle):
    w = fi.cfg4()
    q, k, v = w.qkv()
    lens = list(w.seqlens)
    kp, vp = split(k, lens), split(v, lens)
    ksel = [w.k_sel] * len(lens)
    r = Runner(len(lens), w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", w.total_tokens)
    agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)
    rows = fi.sample_rows(w.seed, lens, 96)
    o, lse = r.sync_exchange(q, k, v, lens, agg)
    oo, ol = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu, rows=rows)
    e = check_close(o[rows], oo, TOL["bf16"], "cfg4 sync exchange")
    check_close(lse[rows], ol, 1e-3, "cfg4 sync exchange lse")
    assert e / np.abs(oo).max() < 0.05


# ---------------------------------------------------------------------------------------------
# a block in which only some participants exchange KV (adaptive aggregation): the others stay local
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 2, 128), ("f32", 4, 2, 64)])
def test_block_with_a_subset_of_participants_exchanging(oracle, dtype, hq, hkv, d):
    lens = [130, 70, 200, 45]
    off = np.concatenate([[0], np.cumsum(lens)])
    q, k, v = gen(61, lens, hq, hkv, d, dtype)
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(len(lens), hq, hkv, d, dtype, sum(lens))
    o_loc, lse_loc = r.local(q, k, v, lens)
    oo_loc, ol_loc = oracle.local(q, k, v, lens)
    for members in ([0, 2], [1, 2, 3], [3]):
        ksel = [lens[n] if n in members else 0 for n in range(len(lens))]      # members send every row
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
        rows = np.concatenate([np.arange(off[n], off[n + 1]) for n in members]).astype(np.int32)
        tc0 = r.ctx.tensor_core_launch_count()
        o, lse = r.sync(q[rows], agg["k_agg"], agg["v_agg"], agg["kv_pos"], q_pos=rows, head_major=True)
        if dtype == "bf16" and sum(ksel) > 0:
            assert r.ctx.tensor_core_launch_count() == tc0 + 1   # the members' rows run on the tensor-core kernel
        oo, ol = oracle.sync(q[rows], ka, va, kv_pos=pos, q_pos=rows, kv_head_major=True)
        check_close(o, oo, TOL[dtype], "subset exchange %s" % members)
        check_close(lse, ol, LSE_TOL[dtype], "subset exchange lse %s" % members)
        rest = np.setdiff1d(np.arange(sum(lens)), rows)
        check_close(o_loc[rest], oo_loc[rest], TOL[dtype], "subset exchange, local rows %s" % members)
    # a participant that exchanges with nobody else computes its local attention
    n0 = np.arange(off[3], off[4])
    check_close(o, oo_loc[n0], TOL[dtype], "lone member equals local")


# ---------------------------------------------------------------------------------------------
# sparse local attention: every participant keeps a seeded sample of its tokens
# ---------------------------------------------------------------------------------------------
def test_sparse_local_attention_on_sampled_tokens(oracle):
    lens = [300, 129, 515]
    hq, hkv, d = 8, 2, 128
    q, k, v = gen(71, lens, hq, hkv, d, "bf16")
    off = np.concatenate([[0], np.cumsum(lens)])
    rng = np.random.default_rng(71)
    keep = [np.sort(rng.choice(n, size=(n + 1) // 2, replace=False)) + off[i] for i, n in enumerate(lens)]
    rows = np.concatenate(keep)
    kept = [len(x) for x in keep]
    r = Runner(len(lens), hq, hkv, d, "bf16", sum(lens))
    o, lse = r.local(q[rows], k[rows], v[rows], kept)
    oo, ol = oracle.local(q[rows], k[rows], v[rows], kept)
    check_close(o, oo, TOL["bf16"], "sparse local")
    check_close(lse, ol, 1e-3, "sparse local lse")


# ---------------------------------------------------------------------------------------------
# decode
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64), ("bf16", 64)])
def test_decode_small(oracle, dtype, d):
    n, cap, hq, hkv = 3, 200, 8, 2
    w = fi.Workload("d", 12, (cap,) * n, hq, hkv, d, dtype)
    _, k, v = w.qkv()
    q = w.decode_q(0)
    kc, vc = k.reshape(n, cap, hkv, d), v.reshape(n, cap, hkv, d)
    r = Runner(n, hq, hkv, d, dtype, n * cap)
    for lens in ([200, 200, 200], [1, 77, 130], [0, 200, 5]):
        o, lse = r.decode(q, kc, vc, lens, False, max_kv_len=cap)
        oo, ol = oracle.decode(q, kc, vc, lens, False)
        check_close(o, oo, TOL[dtype], "decode local %s" % lens)
        check_close(lse, ol, LSE_TOL[dtype], "decode local lse")
    for T in (600, 333, 1):
        o, lse = r.decode(q, k, v, [T], True, max_kv_len=600)
        oo, ol = oracle.decode(q, k, v, [T], True)
        check_close(o, oo, TOL[dtype], "decode sync %d" % T)
        check_close(lse, ol, LSE_TOL[dtype], "decode sync lse")


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_decode_sync_block_with_private_suffix(oracle, dtype, d):
    """Sync-block decode when every participant has generated tokens of its own after the shared
    global cache: attention over the union = sync decode over the global cache, local decode over
    the private suffix, merged by their log-sum-exps."""
    n, T, cap, hq, hkv = 4, 700, 40, 8, 2
    _, kg, vg = fi.Workload("dg", 51, (T,), hq, hkv, d, dtype).qkv()
    ws = fi.Workload("dx", 52, (cap,) * n, hq, hkv, d, dtype)
    _, ks, vs = ws.qkv()
    q = ws.decode_q(0)
    ksc, vsc = ks.reshape(n, cap, hkv, d), vs.reshape(n, cap, hkv, d)
    r = Runner(n, hq, hkv, d, dtype, max(T, n * cap))
    for sfx in ([40, 0, 7, 1], [0, 0, 0, 0]):
        o_g, lse_g = r.decode(q, kg, vg, [T], True, max_kv_len=T)
        o_s, lse_s = r.decode(q, ksc, vsc, sfx, False, max_kv_len=cap)
        o, lse = r.merge(o_g, lse_g, o_s, lse_s)
        cat_k = np.concatenate([np.broadcast_to(kg, (n,) + kg.shape), ksc], axis=1)
        cat_v = np.concatenate([np.broadcast_to(vg, (n,) + vg.shape), vsc], axis=1)
        # the suffix of participant i follows the T global rows directly only when it is read as rows
        # T .. T + sfx[i] - 1, which is how the concatenated cache is laid out
        oo, ol = oracle.decode(q, cat_k, cat_v, [T + s for s in sfx], False)
        check_close(o, oo, TOL[dtype], "decode with suffix %s" % sfx)
        check_close(lse, ol, LSE_TOL[dtype], "decode with suffix lse %s" % sfx)


def test_decode_logits_growing_and_falling_along_the_cache(oracle):
    """Logits that grow (or fall) by far more than 2^8 from tile to tile and from split to split: the
    exponent reference moves inside a CTA's walk, and the partials that are merged differ by hundreds
    of binades (later or earlier splits carry all the weight)."""
    n, cap, hq, hkv, d = 2, 5000, 8, 2, 128
    w = fi.Workload("dg", 33, (cap,) * n, hq, hkv, d, "bf16")
    _, k, v = w.qkv()
    q = fi.round_to_bf16(np.abs(w.decode_q(0)))
    ramp = (np.arange(n * cap, dtype=np.float32) % cap / 40.0)[:, None, None]
    for kk in (fi.round_to_bf16(np.abs(k) * ramp), fi.round_to_bf16(np.abs(k) * ramp[::-1])):
        kc, vc = kk.reshape(n, cap, hkv, d), v.reshape(n, cap, hkv, d)
        r = Runner(n, hq, hkv, d, "bf16", n * cap)
        o, lse = r.decode(q, kc, vc, [cap, 3777], False, max_kv_len=cap)
        oo, ol = oracle.decode(q, kc, vc, [cap, 3777], False)
        check_close(o, oo, TOL["bf16"], "decode local, ramped logits")
        assert np.abs(lse - ol).max() / np.abs(ol).max() < 1e-3
        o, lse = r.decode(q, kk, v, [n * cap], True, max_kv_len=n * cap)
        oo, ol = oracle.decode(q, kk, v, [n * cap], True)
        check_close(o, oo, TOL["bf16"], "decode sync, ramped logits")
        assert np.abs(lse - ol).max() / np.abs(ol).max() < 1e-3


def test_decode_many_splits_clusters_and_row_chunks(oracle):
    """Long caches: the splits of a (cache, KV head) span several clusters, so the cross-cluster merge
    runs; ragged lengths leave some splits empty; 48 stacked rows per KV head need two row chunks."""
    n, cap, hq, hkv, d = 2, 6000, 8, 2, 128
    w = fi.Workload("dl", 31, (cap,) * n, hq, hkv, d, "bf16")
    _, k, v = w.qkv()
    q = w.decode_q(0)
    kc, vc = k.reshape(n, cap, hkv, d), v.reshape(n, cap, hkv, d)
    r = Runner(n, hq, hkv, d, "bf16", n * cap)
    for lens in ([6000, 3333], [6000, 0], [65, 5999]):
        o, lse = r.decode(q, kc, vc, lens, False, max_kv_len=cap)
        oo, ol = oracle.decode(q, kc, vc, lens, False)
        check_close(o, oo, TOL["bf16"], "decode local %s" % lens)
        check_close(lse, ol, 1e-3, "decode local lse %s" % lens)
    n2 = 12                                            # 12 participants x 4 grouped heads = 48 rows per KV head
    w2 = fi.Workload("ds", 32, (500,) * n2, hq, hkv, d, "bf16")
    _, k2, v2 = w2.qkv()
    q2 = w2.decode_q(0)
    r2 = Runner(n2, hq, hkv, d, "bf16", n2 * 500)
    for T in (6000, 4097):
        o, lse = r2.decode(q2, k2, v2, [T], True, max_kv_len=6000)
        oo, ol = oracle.decode(q2, k2, v2, [T], True)
        check_close(o, oo, TOL["bf16"], "decode sync %d" % T)
        check_close(lse, ol, 1e-3, "decode sync lse %d" % T)



def test_decode_more_sources_than_arrival_counters(oracle):
    """64 participants x 16 KV heads = 1024 (cache, KV head) sources: more than the arrival counters of
    the cross-cluster merge could serve, so every source keeps to one cluster."""
    n, cap, hq, hkv, d = 64, 96, 16, 16, 128
    w = fi.Workload("dm", 34, (cap,) * n, hq, hkv, d, "bf16")
    _, k, v = w.qkv()
    q = w.decode_q(0)
    kc, vc = k.reshape(n, cap, hkv, d), v.reshape(n, cap, hkv, d)
    r = Runner(n, hq, hkv, d, "bf16", n * cap)
    lens = [cap - (i % 7) * 9 for i in range(n)]
    o, lse = r.decode(q, kc, vc, lens, False, max_kv_len=cap)
    oo, ol = oracle.decode(q, kc, vc, lens, False)
    check_close(o, oo, TOL["bf16"], "decode local, 1024 sources")
    check_close(lse, ol, LSE_TOL["bf16"], "decode local lse, 1024 sources")


def test_cfg5_decode_full_size(oracle):
    w = fi.cfg5()
    n, cap, hq, hkv, d = 8, 4096, 32, 8, 128
    _, k, v = w.qkv()
    kc, vc = k.reshape(n, cap, hkv, d), v.reshape(n, cap, hkv, d)
    r = Runner(n, hq, hkv, d, "bf16", n * cap)
    for step in (1, 4):
        q = w.decode_q(step)
        if fi.is_sync_block(step, w.sync_interval):
            o, _ = r.decode(q, k, v, [n * cap], True)
            oo, _ = oracle.decode(q, k, v, [n * cap], True)
        else:
            o, _ = r.decode(q, kc, vc, [cap] * n, False)
            oo, _ = oracle.decode(q, kc, vc, [cap] * n, False)
        err = check_close(o, oo, TOL["bf16"], "cfg5 step %d" % step)
        assert err / np.abs(oo).max() < 0.05


# ---------------------------------------------------------------------------------------------
# full-size configurations, sampled rows (rows are independent, so sampled parity is exact)
# ---------------------------------------------------------------------------------------------
def _full_size_local_sync(oracle, w, n_random, block=0):
    q, k, v = w.qkv(block)
    rows = fi.sample_rows(w.seed, w.seqlens, n_random)
    r = Runner(w.n_participants, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.total_tokens)
    o, lse = r.local(q, k, v, w.seqlens)
    oo, ol = oracle.local(q, k, v, w.seqlens, rows=rows)
    e = check_close(o[rows], oo, TOL[w.dtype], w.name + " local")
    check_close(lse[rows], ol, 1e-3, w.name + " local lse")
    assert e / np.abs(oo).max() < 0.05               # not vacuous: error small relative to max |o|
    agg = r.aggregate(fa().AGG_CONCAT, split(k, w.seqlens), split(v, w.seqlens))
    assert np.array_equal(host(agg["k_agg"]), k) and np.array_equal(host(agg["v_agg"]), v)
    o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"])
    oo, ol = oracle.sync(q, k, v, rows=rows)
    e = check_close(o[rows], oo, TOL[w.dtype], w.name + " sync")
    check_close(lse[rows], ol, 1e-3, w.name + " sync lse")
    assert e / np.abs(oo).max() < 0.05


def test_long_segments_many_kv_tiles_sampled(oracle):
    """One 33 k-token participant next to a short one: 258 KV tiles per query tile at the end of the
    walk, ragged last tile, barrier phases and ring stages wrapping many times; odd group size (3 query
    heads per KV head: the last head pair of a KV head is a single head)."""
    w = fi.Workload("long", 77, (32768 + 77, 131), 6, 2, 128, "bf16")
    _full_size_local_sync(oracle, w, 48)


def test_cfg2_full_size_sampled(oracle):
    _full_size_local_sync(oracle, fi.cfg2(), 256)


def test_cfg2_prescaled_reading_relative_error(oracle):
    """Literal alternative reading of config 2 (elements already divided by sqrt(128)): outputs are
    small, so the bound is relative to max |o|."""
    w = fi.cfg2_prescaled().scaled(seqlens=(512,) * 4)
    q, k, v = w.qkv()
    r = Runner(4, 32, 8, 128, "bf16", w.total_tokens)
    o, _ = r.sync(q, k, v)
    oo, _ = oracle.sync(q, k, v)
    assert np.abs(o - oo).max() / np.abs(oo).max() < 0.02


def test_cfg3_one_block_full_size_sampled(oracle):
    _full_size_local_sync(oracle, fi.cfg3(), 96, block=5)


def test_cfg4_sparse_full_size(oracle):
    w = fi.cfg4()
    q, k, v = w.qkv()
    kp, vp = split(k, w.seqlens), split(v, w.seqlens)
    ksel = [w.k_sel] * w.n_participants
    r = Runner(16, 32, 8, 128, "bf16", w.total_tokens)
    agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel)            # bit-exact indices
    assert np.array_equal(agg["kv_pos"].cpu().numpy(), pos) and np.array_equal(agg["cu_kv"].cpu().numpy(), cu)
    assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va)
    rows = fi.sample_rows(w.seed, w.seqlens, 128)
    o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"], head_major=True)
    oo, ol = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True, rows=rows)
    check_close(o[rows], oo, TOL["bf16"], "cfg4 sparse sync")
    check_close(lse[rows], ol, 1e-3, "cfg4 sparse sync lse")


# ---------------------------------------------------------------------------------------------
# C-ABI argument validation: rejected on the host, nothing launched, nothing faults
# ---------------------------------------------------------------------------------------------
def test_invalid_arguments_are_rejected():
    m = fa()
    r = Runner(2, 4, 2, 128, "bf16", 64)
    q = torch.zeros((64, 4, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros_like(q)
    before = r.ctx.launch_count()
    with pytest.raises(m.FedAttnError) as e:
        m.fedattn_local(r.ctx, r.shape, q, kv, kv, [0, 40, 30], o)            # non-monotone offsets
    assert e.value.code == 1
    with pytest.raises(m.FedAttnError):
        m.fedattn_local(r.ctx, r.shape, q, kv, kv, [1, 40, 64], o)            # cu[0] != 0
    with pytest.raises(m.FedAttnError):
        m.fedattn_local(r.ctx, r.shape, None, kv, kv, [0, 40, 64], o)         # null pointer
    with pytest.raises(m.FedAttnError):
        m.fedattn_local(r.ctx, m.Shape(2, 4, 3, 128, m.BF16), q, kv, kv, [0, 40, 64], o)   # Hq % Hkv
    with pytest.raises(m.FedAttnError):
        m.fedattn_aggregate_kv(r.ctx, r.shape, m.AGG_TOPK_KNORM, [kv[:40], kv[40:]], [kv[:40], kv[40:]], [40, 24],
                               [41, 0], None, kv, kv, None, None, None)       # k_sel > L_n
    with pytest.raises(m.FedAttnError):
        m.fedattn_aggregate_kv(r.ctx, r.shape, 7, [kv[:40], kv[40:]], [kv[:40], kv[40:]], [40, 24], None, None,
                               kv, kv, None, None, None)                      # unknown mode
    with pytest.raises(m.FedAttnError):
        m.fedattn_sync(r.ctx, r.shape, q, None, kv, kv, None, -1, False, o)   # negative total_kv
    with pytest.raises(m.FedAttnError):
        m.fedattn_decode(r.ctx, r.shape, 3, q[:2], kv, kv, 0, torch.zeros(2, dtype=torch.int32, device="cuda"), 8,
                         o[:2])                                               # unknown decode mode
    lse = torch.zeros((64, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(m.FedAttnError):
        m.fedattn_sync_remote(r.ctx, r.shape, q, [0, 40, 30], kv, kv, None, 64, False, o, lse)   # non-monotone offsets
    with pytest.raises(m.FedAttnError):
        m.fedattn_merge(r.ctx, r.shape, -1, o, lse, o, lse, o, lse)           # negative row count
    with pytest.raises(m.FedAttnError):
        m.fedattn_merge(r.ctx, r.shape, 64, o, None, o, lse, o, lse)          # a partial result without its lse
    assert r.ctx.launch_count() == before and r.poll() == 0
    m.fedattn_local(r.ctx, r.shape, q, kv, kv, [0, 40, 64], o)                # still usable
    assert r.poll() == 0 and r.ctx.launch_count() > before


# ---------------------------------------------------------------------------------------------
# bounded waits: a wait that runs out is reported, nothing traps, the context stays usable
# ---------------------------------------------------------------------------------------------
def test_wait_timeout_is_reported_and_the_poll_and_repeat_protocol(oracle):
    """The library's own wait routine, run on a barrier that nothing signals with a limit of a few
    polls, gives up, raises status 5 and returns.  Attention calls enqueued before the status is
    polled do no work (outputs untouched); after the poll the same call gives the right result."""
    lens = [150, 130]
    q, k, v = gen(91, lens, 4, 2, 128, "bf16")
    r = Runner(2, 4, 2, 128, "bf16", sum(lens))
    m = fa()
    cu = [0, 150, 280]
    qd, kd, vd = dev(q, "bf16"), dev(k, "bf16"), dev(v, "bf16")
    o = torch.full_like(qd, 7.0)
    r.ctx.selftest_wait_timeout(16)
    m.fedattn_local(r.ctx, r.shape, qd, kd, vd, cu, o)          # enqueued behind the unpolled timeout
    assert r.poll() == 5
    assert torch.all(o == 7.0)                                  # skipped: outputs untouched
    assert r.poll() == 0                                        # the poll cleared the status
    m.fedattn_local(r.ctx, r.shape, qd, kd, vd, cu, o)
    assert r.poll() == 0
    check_close(host(o), oracle.local(q, k, v, lens)[0], TOL["bf16"], "local after a polled timeout")
    with pytest.raises(m.FedAttnError):
        r.ctx.selftest_wait_timeout(0)                          # limit out of range: rejected on the host


# ---------------------------------------------------------------------------------------------
# seeded random shapes: every bf16 head_dim-128 path on segment lengths around the tile edges
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_seeded_random_shapes_prefill_paths(oracle, seed):
    """Participants, segment lengths (0, 1, around 32 / 128 / 256 / 512), group sizes (1..4, odd ones
    included) and kept counts drawn from a seeded generator; local, dense sync, per-head and token-level
    selection, sync over the sparse aggregate, the exchange block, the indexed gather with the selected
    indices, and a shuffled row order through explicit positions, all against the oracle."""
    rng = np.random.default_rng(seed)
    for case in range(6):
        n = int(rng.integers(1, 7))
        lens = [int(x) for x in rng.choice([0, 1, 5, 31, 32, 33, 64, 100, 127, 128, 129, 200, 256, 257, 300, 384, 513], size=n)]
        if sum(lens) == 0:
            lens[0] = 7
        hkv = int(rng.choice([1, 2, 4])); hq = hkv * int(rng.choice([1, 2, 3, 4]))
        causal = bool(rng.integers(0, 4) != 0)
        q, k, v = gen(int(rng.integers(1, 10**6)), lens, hq, hkv, 128, "bf16")
        what = "seed %d case %d lens %s hq %d hkv %d causal %s: " % (seed, case, lens, hq, hkv, causal)
        r = Runner(n, hq, hkv, 128, "bf16", sum(lens), causal=causal)
        o, lse = r.local(q, k, v, lens)
        oo, ol = oracle.local(q, k, v, lens, causal=causal)
        check_close(o, oo, TOL["bf16"], what + "local"); check_close(lse, ol, LSE_TOL["bf16"], what + "local lse")
        o, lse = r.sync(q, k, v)
        oo, ol = oracle.sync(q, k, v, causal=causal)
        check_close(o, oo, TOL["bf16"], what + "sync"); check_close(lse, ol, LSE_TOL["bf16"], what + "sync lse")
        kp, vp = split(k, lens), split(v, lens)
        ksel = [int(rng.integers(0, x + 1)) for x in lens]
        agg = r.aggregate(fa().AGG_TOPK_KNORM, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
        assert agg["status"] == 0 and np.array_equal(agg["sel_idx"].cpu().numpy(), sel), what + "selection"
        assert np.array_equal(host(agg["k_agg"]), ka) and np.array_equal(host(agg["v_agg"]), va), what + "rows"
        if sum(ksel) > 0:
            o, lse = r.sync(q, agg["k_agg"], agg["v_agg"], agg["kv_pos"], head_major=True)
            oo, ol = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True, causal=causal)
            check_close(o, oo, TOL["bf16"], what + "sparse sync"); check_close(lse, ol, LSE_TOL["bf16"], what + "sparse sync lse")
            o, lse = r.sync_exchange(q, k, v, lens, agg)
            oo, ol = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu, causal=causal)
            check_close(o, oo, TOL["bf16"], what + "exchange"); check_close(lse, ol, LSE_TOL["bf16"], what + "exchange lse")
            again = r.aggregate(fa().AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)
            assert again["status"] == 0 and np.array_equal(host(again["k_agg"]), ka), what + "indexed"
            assert np.array_equal(again["kv_pos"].cpu().numpy(), pos), what + "indexed positions"
        agg = r.aggregate(fa().AGG_TOPK_TOKEN, kp, vp, ksel)
        ka, va, pos, cu, sel = oracle.aggregate_topk_token(kp, vp, ksel)
        assert np.array_equal(agg["sel_idx"].cpu().numpy(), sel) and np.array_equal(host(agg["k_agg"]), ka), what + "token"
        if causal and sum(lens) > 1:
            perm = rng.permutation(sum(lens))
            o, lse = r.sync(q[perm], k[perm], v[perm], kv_pos=perm.astype(np.int32), q_pos=perm.astype(np.int32))
            oo, ol = oracle.sync(q, k, v, causal=True)
            check_close(o, oo[perm], TOL["bf16"], what + "shuffled rows"); check_close(lse, ol[perm], LSE_TOL["bf16"], what + "shuffled rows lse")


@pytest.mark.parametrize("seed", [1, 2])
def test_seeded_random_shapes_decode(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    for case in range(8):
        n = int(rng.integers(1, 9)); cap = int(rng.choice([1, 17, 64, 65, 200, 512, 1000, 3000]))
        hkv = int(rng.choice([1, 2, 8])); hq = hkv * int(rng.choice([1, 2, 4]))
        w = fi.Workload("d", int(rng.integers(1, 10**6)), (cap,) * n, hq, hkv, 128, "bf16")
        _, k, v = w.qkv()
        q = w.decode_q(0)
        kc, vc = k.reshape(n, cap, hkv, 128), v.reshape(n, cap, hkv, 128)
        lens = [int(rng.integers(0, cap + 1)) for _ in range(n)]
        T = int(rng.integers(1, n * cap + 1))
        what = "seed %d case %d n %d cap %d hq %d hkv %d: " % (seed, case, n, cap, hq, hkv)
        r = Runner(n, hq, hkv, 128, "bf16", n * cap)
        o, lse = r.decode(q, kc, vc, lens, False, max_kv_len=cap)
        oo, ol = oracle.decode(q, kc, vc, lens, False)
        check_close(o, oo, TOL["bf16"], what + "local"); check_close(lse, ol, LSE_TOL["bf16"], what + "local lse")
        o, lse = r.decode(q, k, v, [T], True, max_kv_len=n * cap)
        oo, ol = oracle.decode(q, k, v, [T], True)
        check_close(o, oo, TOL["bf16"], what + "sync"); check_close(lse, ol, LSE_TOL["bf16"], what + "sync lse")


def test_indexed_gather_empty_in_place_and_sixty_four_participants(oracle):
    """INDEXED aggregation at its edges: nothing kept at all; the kept indices given and returned in the
    same buffer, three calls in a row; the largest participant count the interface takes."""
    m = fa()
    lens = [40, 7, 300]
    _, k, v = gen(5, lens, 4, 2, 128, "bf16")
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(3, 4, 2, 128, "bf16", sum(lens))
    agg = r.aggregate(m.AGG_INDEXED, kp, vp, [0, 0, 0], sel_idx_in=np.zeros((2, 0), dtype=np.int32))
    assert agg["status"] == 0 and list(agg["cu_kv"].cpu().numpy()) == [0, 0, 0, 0]
    ksel = [10, 7, 100]
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    T = sum(ksel)
    kd, vd = [dev(x, "bf16") for x in kp], [dev(x, "bf16") for x in vp]
    sel_d = torch.from_numpy(sel.astype(np.int32)).cuda()
    for _ in range(3):
        k2 = torch.zeros((2, T, 128), dtype=torch.bfloat16, device="cuda"); v2 = torch.zeros_like(k2)
        p2 = torch.zeros((2, T), dtype=torch.int32, device="cuda"); c2 = torch.zeros(4, dtype=torch.int32, device="cuda")
        m.fedattn_aggregate_kv(r.ctx, r.shape, m.AGG_INDEXED, kd, vd, lens, ksel, sel_d, k2, v2, p2, c2, sel_d)
        assert r.poll() == 0
        assert np.array_equal(host(k2), ka) and np.array_equal(host(v2), va)
        assert np.array_equal(p2.cpu().numpy(), pos) and np.array_equal(c2.cpu().numpy(), cu)
        assert np.array_equal(sel_d.cpu().numpy(), sel)
    lens = [16] * 64
    _, k, v = gen(6, lens, 2, 1, 128, "bf16")
    kp, vp = split(k, lens), split(v, lens)
    r = Runner(64, 2, 1, 128, "bf16", sum(lens))
    ksel = [4] * 64
    ka, va, pos, cu, sel = oracle.aggregate_topk(kp, vp, ksel)
    a1 = r.aggregate(m.AGG_TOPK_KNORM, kp, vp, ksel)
    a2 = r.aggregate(m.AGG_INDEXED, kp, vp, ksel, sel_idx_in=sel)
    assert a1["status"] == 0 and a2["status"] == 0
    assert np.array_equal(a1["sel_idx"].cpu().numpy(), sel) and np.array_equal(host(a1["k_agg"]), ka)
    assert np.array_equal(host(a2["k_agg"]), ka) and np.array_equal(host(a2["v_agg"]), va)
    assert np.array_equal(a2["kv_pos"].cpu().numpy(), pos)
