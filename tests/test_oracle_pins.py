"""Pins for the fp64 CPU oracle: each test checks it against something the paper or the
mathematics fixes (closed forms, textbook special cases, a library routine, brute force),
never against the CUDA path.  Runs without a GPU."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import fedattn_inputs as fi

RNG = np.random.default_rng(1234)


def randn(*shape):
    return RNG.standard_normal(shape)


# ----------------------------------------------------------------------------------------------
# brute force written separately from the row-wise oracle: nested loops, math.exp, python floats
# ----------------------------------------------------------------------------------------------
def brute_attention(q, K, V, allowed_fn, scale):
    """q [Lq,Hq,d]; K,V given by accessor (j, kvh) -> row; allowed_fn(i, kvh) -> list of j."""
    Lq, Hq, d = q.shape
    o = np.zeros((Lq, Hq, d))
    lse = np.full((Lq, Hq), -np.inf)
    for i in range(Lq):
        for h in range(Hq):
            js, kvh = allowed_fn(i, h)
            if not js:
                continue
            logits = [scale * sum(float(q[i, h, c]) * float(K(j, kvh)[c]) for c in range(d)) for j in js]
            m = max(logits)
            w = [math.exp(x - m) for x in logits]
            z = sum(w)
            for t, j in enumerate(js):
                for c in range(d):
                    o[i, h, c] += w[t] / z * float(V(j, kvh)[c])
            lse[i, h] = m + math.log(z)
    return o, lse


def test_offsets_bruteforce(oracle):
    for _ in range(20):
        n = int(RNG.integers(1, 17))
        lens = RNG.integers(0, 5000, size=n)
        off = oracle.offsets(lens)
        assert off[0] == 0 and off[-1] == lens.sum()
        for i in range(n):
            assert off[i] == sum(int(x) for x in lens[:i])
        # disjoint cover of 0..L-1 in participant order
        cover = np.concatenate([np.arange(off[i], off[i + 1]) for i in range(n)]) if lens.sum() else np.array([])
        assert np.array_equal(cover, np.arange(lens.sum()))


@pytest.mark.parametrize("causal", [True, False])
def test_local_bruteforce_tiny(oracle, causal):
    lens = [3, 1, 5]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    off = np.concatenate([[0], np.cumsum(lens)])
    scale = 1.0 / math.sqrt(d)

    def allowed(i, h):
        n = max(x for x in range(len(lens)) if off[x] <= i)
        hi = i if causal else off[n + 1] - 1
        return list(range(off[n], hi + 1)), h // (Hq // Hkv)

    bo, bl = brute_attention(q, lambda j, kh: k[j, kh], lambda j, kh: v[j, kh], allowed, scale)
    o, lse = oracle.local(q, k, v, lens, causal=causal)
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - bl).max() < 1e-12


def test_local_n1_equals_library_causal_attention(oracle):
    """N=1 reduces FedAttn to centralised attention (Sec. VI, discussion of the number of
    participants); cross-checked against torch's fp64 scaled_dot_product_attention."""
    L, Hq, Hkv, d = 37, 4, 2, 8
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    o, _ = oracle.local(q, k, v, [L])
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(k, Hq // Hkv, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, Hq // Hkv, axis=1)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.abs(o - ref).max() < 1e-12
    # bidirectional variant against the same routine without the mask
    o2, _ = oracle.local(q, k, v, [L], causal=False)
    ref2 = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0].permute(1, 0, 2).numpy()
    assert np.abs(o2 - ref2).max() < 1e-12


def test_local_is_block_diagonal(oracle):
    lens = [5, 9, 1, 7]
    L, Hq, Hkv, d = sum(lens), 2, 2, 8
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    o, lse = oracle.local(q, k, v, lens)
    off = 0
    for ln in lens:
        oi, li = oracle.local(q[off:off + ln], k[off:off + ln], v[off:off + ln], [ln])
        assert np.array_equal(o[off:off + ln], oi) and np.array_equal(lse[off:off + ln], li)
        off += ln
    # changing another participant's K/V must not change this participant's output
    k2, v2 = k.copy(), v.copy()
    k2[:5] += 3.0
    v2[:5] -= 2.0
    o2, _ = oracle.local(q, k2, v2, lens)
    assert np.array_equal(o[5:], o2[5:])


def test_softmax_rows_sum_to_one_and_scale_convention(oracle):
    """V = 1 returns exactly the row sum of the attention weights; scale defaults to
    1/sqrt(head_dim)."""
    lens = [6, 4]
    L, H, d = 10, 2, 16
    q, k = randn(L, H, d), randn(L, H, d)
    o, _ = oracle.local(q, k, np.ones((L, H, d)), lens)
    assert np.abs(o - 1.0).max() < 1e-12
    v = randn(L, H, d)
    a, _ = oracle.local(q, k, v, lens)
    b, _ = oracle.local(q, k, v, lens, scale=1.0 / math.sqrt(d))
    c, _ = oracle.local(q * 2.0, k, v, lens, scale=0.5 / math.sqrt(d))
    assert np.array_equal(a, b) and np.abs(a - c).max() < 1e-12


@pytest.mark.parametrize("mode", ["local", "sync"])
def test_equal_keys_closed_form_pins_mask_boundaries(oracle, mode):
    """All keys equal => uniform weights => o_i is the arithmetic mean of V over the allowed
    set and lse_i = scale * q_i.k + ln|allowed|; checks every first/last allowed index."""
    lens = [4, 1, 6, 3]
    L, Hq, Hkv, d = sum(lens), 2, 1, 4
    off = np.concatenate([[0], np.cumsum(lens)])
    q, v = randn(L, Hq, d), randn(L, Hkv, d)
    kvec = randn(d)
    k = np.broadcast_to(kvec, (L, Hkv, d)).copy()
    scale = 1.0 / math.sqrt(d)
    if mode == "local":
        o, lse = oracle.local(q, k, v, lens)
    else:
        o, lse = oracle.sync(q, k, v)
    for i in range(L):
        n = max(x for x in range(len(lens)) if off[x] <= i)
        lo = off[n] if mode == "local" else 0
        mean = v[lo:i + 1, 0].mean(axis=0)
        for h in range(Hq):
            assert np.abs(o[i, h] - mean).max() < 1e-12
            assert abs(lse[i, h] - (scale * q[i, h] @ kvec + math.log(i + 1 - lo))) < 1e-12


def test_sync_dense_equals_centralised_attention(oracle):
    """Sync at every block (H=1) is centralised attention: local queries over the
    concatenated KV equal the N=1 result on the concatenated sequence (Remark after
    Corollary 1; appendix on CenAttn)."""
    lens = [7, 3, 11]
    L, Hq, Hkv, d = sum(lens), 4, 2, 8
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    parts_k = np.split(k, np.cumsum(lens)[:-1])
    parts_v = np.split(v, np.cumsum(lens)[:-1])
    k_agg, v_agg, kv_pos, cu = oracle.aggregate_concat(parts_k, parts_v)
    o_sync, lse_sync = oracle.sync(q, k_agg, v_agg, kv_pos=kv_pos)
    o_cen, lse_cen = oracle.local(q, k, v, [L])
    assert np.abs(o_sync - o_cen).max() < 1e-13 and np.abs(lse_sync - lse_cen).max() < 1e-13
    # per-participant calls with explicit positions give the same rows
    off = 0
    for ln in lens:
        oi, _ = oracle.sync(q[off:off + ln], k_agg, v_agg, kv_pos=kv_pos, q_pos=np.arange(off, off + ln))
        assert np.abs(oi - o_cen[off:off + ln]).max() < 1e-13
        off += ln


def test_sync_tends_to_local_when_remote_logits_vanish(oracle):
    """Remote logits pushed to -700 or lower make the inter-participant weights vanish:
    global attention then equals local attention."""
    lens = [5, 8, 4]
    L, H, d = sum(lens), 2, 6
    q, k, v = randn(L, H, d), randn(L, H, d), randn(L, H, d)
    part = np.repeat(np.arange(len(lens)), lens)
    B = 1.0e4
    q[:, :, 0] = 1.0
    k[:, :, 0] = B * part[:, None]          # own keys exceed earlier participants' by >= B
    o_s, _ = oracle.sync(q, k, v, scale=1.0)
    o_l, _ = oracle.local(q, k, v, lens, scale=1.0)
    assert np.abs(o_s - o_l).max() < 1e-12


def test_aggregate_concat_is_memcpy(oracle):
    lens = [3, 0, 5, 1]
    Hkv, d = 2, 4
    ks = [randn(n, Hkv, d) for n in lens]
    vs = [randn(n, Hkv, d) for n in lens]
    k_agg, v_agg, kv_pos, cu = oracle.aggregate_concat(ks, vs)
    assert k_agg.tobytes() == np.concatenate(ks).tobytes()
    assert v_agg.tobytes() == np.concatenate(vs).tobytes()
    assert np.array_equal(kv_pos, np.arange(sum(lens)))
    assert np.array_equal(cu, [0, 3, 3, 8, 9])


def rank_select(scores, k):
    """Independent selector: token i is kept iff fewer than k tokens beat it, where j beats i
    when score_j > score_i, or they tie and j < i."""
    n = len(scores)
    keep = []
    for i in range(n):
        beat = sum(1 for j in range(n) if scores[j] > scores[i] or (scores[j] == scores[i] and j < i))
        if beat < k:
            keep.append(i)
    return keep


def test_topk_bruteforce_and_ties(oracle):
    ln, Hkv, d = 40, 3, 8
    kp = fi.round_to_bf16(randn(ln, Hkv, d).astype(np.float32)).astype(np.float64)
    kp[7] = kp[3]                      # planted duplicates
    kp[21] = kp[3]
    kp[30, 1] = -kp[5, 1]              # same norm, different sign
    for ksel in [0, 1, 5, 13, 39, 40]:
        sel, scores = oracle.topk_knorm(kp, ksel, return_scores=True)
        for h in range(Hkv):
            s = [sum(float(x) * float(x) for x in kp[j, h]) for j in range(ln)]
            assert np.array_equal(scores[h], np.array(s))
            assert list(sel[h]) == rank_select(s, ksel)


def test_topk_constructed_norms(oracle):
    ln, Hkv, d = 16, 1, 4
    kp = np.zeros((ln, Hkv, d))
    kp[:, 0, 0] = np.arange(ln, 0, -1)          # strictly decreasing => first k
    assert list(oracle.topk_knorm(kp, 5)[0]) == [0, 1, 2, 3, 4]
    kp[:, 0, 0] = 1.0                           # all equal => first k by the tie rule
    assert list(oracle.topk_knorm(kp, 5)[0]) == [0, 1, 2, 3, 4]
    kp[:, 0, 0] = np.arange(1, ln + 1)          # increasing => last k, ascending
    assert list(oracle.topk_knorm(kp, 3)[0]) == [13, 14, 15]
    kp[:, 0, 0] = [5, 9, 9, 1, 9, 2, 9, 0, 0, 0, 0, 0, 0, 0, 0, 0]   # duplicates straddle k-th place
    assert list(oracle.topk_knorm(kp, 2)[0]) == [1, 2]
    assert list(oracle.topk_knorm(kp, 3)[0]) == [1, 2, 4]
    # square of the norm, not the signed sum
    kp[:, 0, :] = 0.0
    kp[2, 0] = [-3, 0, 0, 0]
    kp[9, 0] = [1, 1, 1, 1]
    assert list(oracle.topk_knorm(kp, 1)[0]) == [2]


def test_token_level_selection_bruteforce_and_special_cases(oracle):
    """Token-level selection: one score per token over all KV heads, the same tokens for every head."""
    lens = [9, 6, 7]
    Hkv, d = 3, 4
    ks = [fi.round_to_bf16(randn(n, Hkv, d).astype(np.float32)).astype(np.float64) for n in lens]
    vs = [randn(n, Hkv, d) for n in lens]
    ks[0][4] = ks[0][1]                          # a tie between tokens 1 and 4
    ks[2][5] = ks[2][0][::-1]                    # heads permuted: the same terms in another order
    off = np.concatenate([[0], np.cumsum(lens)])
    ksel = [4, 0, 3]
    k_agg, v_agg, kv_pos, cu, sel = oracle.aggregate_topk_token(ks, vs, ksel)
    assert k_agg.shape == (7, Hkv, d) and kv_pos.shape == (7,) and np.array_equal(cu, [0, 4, 4, 7])
    at = 0
    for n, kk in enumerate(ksel):
        # nested-loop score in memory order (head, then channel), python floats = the fp64 chain
        score = []
        for j in range(lens[n]):
            acc = 0.0
            for h in range(Hkv):
                for c in range(d):
                    acc = acc + float(ks[n][j, h, c]) * float(ks[n][j, h, c])
            score.append(acc)
        want = rank_select(score, kk)
        assert list(sel[at:at + kk]) == want
        for t, j in enumerate(want):
            assert np.array_equal(k_agg[at + t], ks[n][j]) and np.array_equal(v_agg[at + t], vs[n][j])
            assert kv_pos[at + t] == off[n] + j
        at += kk
    # one KV head: token-level and per-head selection coincide
    k1 = [x[:, :1] for x in ks]; v1 = [x[:, :1] for x in vs]
    a = oracle.aggregate_topk_token(k1, v1, ksel)
    b = oracle.aggregate_topk(k1, v1, ksel)
    assert np.array_equal(a[0], b[0][0][:, None, :]) and np.array_equal(a[2], b[2][0]) and np.array_equal(a[4], b[4][0])
    # every token kept: the concatenation
    ka, va, pos, cu2 = oracle.aggregate_concat(ks, vs)
    k_all, v_all, pos_all, _, _ = oracle.aggregate_topk_token(ks, vs, lens)
    assert np.array_equal(k_all, ka) and np.array_equal(v_all, va) and np.array_equal(pos_all, pos)


def test_sparse_aggregation_layout_and_special_cases(oracle):
    lens = [6, 4, 5]
    Hkv, d = 2, 4
    ks = [randn(n, Hkv, d) for n in lens]
    vs = [randn(n, Hkv, d) for n in lens]
    off = np.concatenate([[0], np.cumsum(lens)])
    ksel = [2, 0, 3]
    k_agg, v_agg, kv_pos, cu, sel = oracle.aggregate_topk(ks, vs, ksel)
    assert np.array_equal(cu, [0, 2, 2, 5]) and sel.shape == (Hkv, 5)
    for h in range(Hkv):
        for n in range(3):
            for t in range(ksel[n]):
                j = sel[h, cu[n] + t]
                assert np.array_equal(k_agg[h, cu[n] + t], ks[n][j, h])
                assert np.array_equal(v_agg[h, cu[n] + t], vs[n][j, h])
                assert kv_pos[h, cu[n] + t] == off[n] + j
            seg = sel[h, cu[n]:cu[n + 1]]
            assert np.all(np.diff(seg) > 0)
    # k_n = L_n keeps everything: equals dense concatenation, head-major
    k_all, v_all, pos_all, cu_all, sel_all = oracle.aggregate_topk(ks, vs, lens)
    kc, vc, pc, cc = oracle.aggregate_concat(ks, vs)
    assert np.array_equal(k_all, kc.transpose(1, 0, 2)) and np.array_equal(v_all, vc.transpose(1, 0, 2))
    assert np.array_equal(pos_all, np.broadcast_to(pc, (Hkv, sum(lens)))) and np.array_equal(cu_all, cc)


def test_sparse_sync_special_cases_and_bruteforce(oracle):
    lens = [4, 3, 5]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    cuts = np.cumsum(lens)[:-1]
    ks, vs = np.split(k, cuts), np.split(v, cuts)
    dense, dense_lse = oracle.sync(q, k, v)
    # every key kept => dense result
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, lens)
    o, lse = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True)
    assert np.abs(o - dense).max() < 1e-13 and np.abs(lse - dense_lse).max() < 1e-13
    # excluded participant (empty L'_n) => sync over the others, positions kept
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, [4, 0, 5])
    o, _ = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True)
    keep = np.r_[0:4, 7:12]
    o_ref, _ = oracle.sync(q, k[keep], v[keep], kv_pos=keep)
    assert np.abs(o - o_ref).max() < 1e-13
    # brute force incl. rows whose allowed set is empty (first participant excluded)
    ksel = [0, 2, 3]
    ka, va, pos, cu, sel = oracle.aggregate_topk(ks, vs, ksel)
    o, lse = oracle.sync(q, ka, va, kv_pos=pos, kv_head_major=True)
    g = Hq // Hkv

    def allowed(i, h):
        return [j for j in range(ka.shape[1]) if pos[h // g, j] <= i], h // g

    bo, bl = brute_attention(q, lambda j, kh: ka[kh, j], lambda j, kh: va[kh, j], allowed, 1 / math.sqrt(d))
    assert np.abs(o - bo).max() < 1e-12
    assert np.all(o[:4] == 0.0) and np.all(np.isneginf(lse[:4]))
    fin = np.isfinite(bl)
    assert np.array_equal(fin, np.isfinite(lse)) and np.abs(lse[fin] - bl[fin]).max() < 1e-12


# ----------------------------------------------------------------------------------------------
# sync block with sparse KV exchange (own segment complete, remote keys sparsified)
# ----------------------------------------------------------------------------------------------
def lse_merge(o_a, lse_a, o_b, lse_b):
    """Attention over a disjoint union of key sets from the two partial results (closed form)."""
    m = np.maximum(lse_a, lse_b)
    m = np.where(np.isfinite(m), m, 0.0)
    wa, wb = np.exp(lse_a - m), np.exp(lse_b - m)
    z = wa + wb
    o = (o_a * wa[..., None] + o_b * wb[..., None]) / np.where(z > 0, z, 1.0)[..., None]
    return o, m + np.log(z)


def test_sync_exchange_special_cases(oracle):
    lens = [4, 3, 5]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    cuts = np.cumsum(lens)[:-1]
    ks, vs = np.split(k, cuts), np.split(v, cuts)
    # every remote key exchanged => the dense sync block (= centralised attention)
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, lens)
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    dense, dense_lse = oracle.sync(q, k, v)
    assert np.abs(o - dense).max() < 1e-13 and np.abs(lse - dense_lse).max() < 1e-13
    # nothing exchanged => the local block
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, [0, 0, 0])
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    loc, loc_lse = oracle.local(q, k, v, lens)
    assert np.abs(o - loc).max() < 1e-13 and np.abs(lse - loc_lse).max() < 1e-13
    # a participant's own exchanged rows must not be counted twice: with only participant 1 sending,
    # participant 1's own rows are unchanged and participant 0 (earlier) sees nothing new
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, [0, 3, 0])
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    assert np.abs(o[:7] - loc[:7]).max() < 1e-13 and np.abs(lse[:7] - loc_lse[:7]).max() < 1e-13
    assert np.abs(o[7:] - loc[7:]).max() > 1e-3


def test_sync_exchange_bruteforce_and_equal_keys(oracle):
    lens = [3, 4, 2, 4]
    L, Hq, Hkv, d = sum(lens), 4, 2, 3
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    off = np.concatenate([[0], np.cumsum(lens)])
    ks, vs = np.split(k, off[1:-1]), np.split(v, off[1:-1])
    ksel = [2, 1, 0, 3]
    ka, va, pos, cu, sel = oracle.aggregate_topk(ks, vs, ksel)
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    g = Hq // Hkv
    T = ka.shape[1]
    seg = np.searchsorted(off, np.arange(L), side="right") - 1

    # brute force over a tagged union: ("l", j) local rows, ("a", t) exchanged rows
    def allowed(i, h):
        n, kvh = seg[i], h // g
        own = [("l", j) for j in range(off[n], i + 1)]
        remote = [("a", t) for t in range(T) if not (cu[n] <= t < cu[n + 1]) and pos[kvh, t] <= i]
        return own + remote, kvh

    K = lambda key, kh: k[key[1], kh] if key[0] == "l" else ka[kh, key[1]]
    V = lambda key, kh: v[key[1], kh] if key[0] == "l" else va[kh, key[1]]
    bo, bl = brute_attention(q, K, V, allowed, 1 / math.sqrt(d))
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - bl).max() < 1e-12
    # all keys equal => uniform weights: o = mean of V over the allowed set, lse = logit + ln |allowed|
    k_eq = np.broadcast_to(randn(1, Hkv, d), (L, Hkv, d)).copy()
    ka2, va2, pos2, cu2 = oracle.aggregate_indexed(np.split(k_eq, off[1:-1]), vs, ksel, sel)
    o, lse = oracle.sync_exchange(q, k_eq, v, lens, ka2, va2, pos2, cu2)
    for i in (0, 2, 3, 6, 8, 9, 12):
        for h in range(Hq):
            keys, kvh = allowed(i, h)
            mean_v = np.mean([V(key, kvh) for key in keys], axis=0)
            logit = float(q[i, h] @ k_eq[0, kvh]) / math.sqrt(d)
            assert np.abs(o[i, h] - mean_v).max() < 1e-12
            assert abs(lse[i, h] - (logit + math.log(len(keys)))) < 1e-12


def test_sync_exchange_is_local_merged_with_remote_only_sync(oracle):
    """The decomposition the CUDA path uses: attention over own keys (local block) and over the
    exchanged keys of earlier participants (a sync call whose query position is the last position
    before the participant's segment), merged through their log-sum-exps."""
    lens = [5, 2, 6, 3]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    off = np.concatenate([[0], np.cumsum(lens)])
    ks, vs = np.split(k, off[1:-1]), np.split(v, off[1:-1])
    ka, va, pos, cu, _ = oracle.aggregate_topk(ks, vs, [3, 1, 4, 2])
    want, want_lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    seg = np.searchsorted(off, np.arange(L), side="right") - 1
    o_l, lse_l = oracle.local(q, k, v, lens)
    o_r, lse_r = oracle.sync(q, ka, va, kv_pos=pos, q_pos=off[seg] - 1, kv_head_major=True)
    o, lse = lse_merge(o_l, lse_l, o_r, lse_r)
    assert np.abs(o - want).max() < 1e-12 and np.abs(lse - want_lse).max() < 1e-12



@pytest.mark.parametrize("ksel", [[2, 1, 0, 3], [3, 4, 2, 4], [0, 0, 0, 0]])
def test_sync_exchange_bidirectional_bruteforce_and_limits(oracle, ksel):
    """causal = 0: a row attends its whole own segment and every exchanged key of the other
    participants (Sec. III-B: attention without the mask).  Brute force over a tagged union; with
    every key exchanged it is bidirectional attention over the whole sequence, with none it is the
    bidirectional local block."""
    lens = [3, 4, 2, 4]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    off = np.concatenate([[0], np.cumsum(lens)])
    ks, vs = np.split(k, off[1:-1]), np.split(v, off[1:-1])
    sel = fi.random_selection(77, lens, ksel, Hkv)
    ka, va, pos, cu = oracle.aggregate_indexed(ks, vs, ksel, sel)
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu, causal=False)
    g, T = Hq // Hkv, ka.shape[1]
    seg = np.searchsorted(off, np.arange(L), side="right") - 1

    def allowed(i, h):
        n = seg[i]
        own = [("l", j) for j in range(off[n], off[n + 1])]
        remote = [("a", t) for t in range(T) if not (cu[n] <= t < cu[n + 1])]
        return own + remote, h // g

    K = lambda key, kh: k[key[1], kh] if key[0] == "l" else ka[kh, key[1]]
    V = lambda key, kh: v[key[1], kh] if key[0] == "l" else va[kh, key[1]]
    bo, bl = brute_attention(q, K, V, allowed, 1 / math.sqrt(d))
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - bl).max() < 1e-12
    if ksel == lens:
        dense, dense_lse = oracle.sync(q, k, v, causal=False)
        assert np.abs(o - dense).max() < 1e-12 and np.abs(lse - dense_lse).max() < 1e-12
    if sum(ksel) == 0:
        loc, loc_lse = oracle.local(q, k, v, lens, causal=False)
        assert np.abs(o - loc).max() < 1e-13 and np.abs(lse - loc_lse).max() < 1e-13
    # the decomposition the CUDA path uses: bidirectional local block merged with a remote-only pass
    o_l, lse_l = oracle.local(q, k, v, lens, causal=False)
    o_r = np.zeros_like(o_l); lse_r = np.full_like(lse_l, -np.inf)
    for n in range(len(lens)):
        keep = np.array([t for t in range(T) if not (cu[n] <= t < cu[n + 1])], dtype=np.int64)
        if len(keep) and lens[n]:
            rows = np.arange(off[n], off[n + 1])
            o_r[rows], lse_r[rows] = oracle.sync(q[rows], ka[:, keep], va[:, keep], kv_head_major=True, causal=False)
    om, lm = lse_merge(o_l, lse_l, o_r, lse_r)
    assert np.abs(om - o).max() < 1e-12 and np.abs(lm - lse).max() < 1e-12


def test_random_selection_feeds_the_exchange_block(oracle):
    """The sparsity-ratio experiment samples the exchanged KV rows at random (Sec. VI): a seeded draw
    per (participant, KV head) goes through the indexed aggregation into the exchange block.  Pinned
    by brute force over the tagged union, by the draw's own invariants, and by the two limits."""
    lens = [5, 3, 6, 4]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    off = np.concatenate([[0], np.cumsum(lens)])
    ks, vs = np.split(k, off[1:-1]), np.split(v, off[1:-1])
    ksel = [2, 1, 3, 2]                                   # ratio 1/2, rounded
    sel = fi.random_selection(5, lens, ksel, Hkv)
    cu = np.concatenate([[0], np.cumsum(ksel)])
    for h in range(Hkv):
        for n in range(len(lens)):
            blk = sel[h, cu[n]:cu[n + 1]]
            assert np.all(np.diff(blk) > 0) and (len(blk) == 0 or (blk[0] >= 0 and blk[-1] < lens[n]))
    assert not np.array_equal(sel[0], sel[1])             # heads draw independently
    assert np.array_equal(sel, fi.random_selection(5, lens, ksel, Hkv))   # seeded
    ka, va, pos, cu2 = oracle.aggregate_indexed(ks, vs, ksel, sel)
    assert np.array_equal(cu2, cu)
    o, lse = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu)
    g, T = Hq // Hkv, ka.shape[1]
    seg = np.searchsorted(off, np.arange(L), side="right") - 1

    def allowed(i, h):
        n, kvh = seg[i], h // g
        own = [("l", j) for j in range(off[n], i + 1)]
        remote = [("r", (m, int(j))) for m in range(len(lens)) if m != n
                  for j in sel[kvh, cu[m]:cu[m + 1]] if off[m] + j <= i]
        return own + remote, kvh

    K = lambda key, kh: k[key[1], kh] if key[0] == "l" else ks[key[1][0]][key[1][1], kh]
    V = lambda key, kh: v[key[1], kh] if key[0] == "l" else vs[key[1][0]][key[1][1], kh]
    bo, bl = brute_attention(q, K, V, allowed, 1 / math.sqrt(d))
    assert np.abs(o - bo).max() < 1e-12 and np.abs(lse - bl).max() < 1e-12
    full = fi.random_selection(5, lens, lens, Hkv)        # ratio 1: every row, i.e. the dense sync block
    ka, va, pos, cu3 = oracle.aggregate_indexed(ks, vs, lens, full)
    dense, dense_lse = oracle.sync(q, k, v)
    o1, l1 = oracle.sync_exchange(q, k, v, lens, ka, va, pos, cu3)
    assert np.abs(o1 - dense).max() < 1e-13 and np.abs(l1 - dense_lse).max() < 1e-13


@pytest.mark.parametrize("kind", ["interleaved", "random", "contiguous"])
def test_general_index_sets_sync_equals_centralised_attention(oracle, kind):
    """Sec. IV-A: the participants hold general ordered index sets L_n of the global sequence.  With
    explicit positions for queries and aggregated keys, syncing reproduces centralised attention on
    the sequence in its global order (the H = 1 reduction), whatever the partition; the concatenated
    kv_pos is then not monotone.  Checked against torch's fp64 causal attention on the re-ordered
    sequence and, for one participant's rows alone, against brute force."""
    lens = [5, 2, 6, 3]
    L, Hq, Hkv, d = sum(lens), 4, 2, 8
    sets = fi.index_sets(9, lens, kind)
    assert np.array_equal(np.sort(np.concatenate(sets)), np.arange(L))
    pos = np.concatenate(sets).astype(np.int32)            # packed row r holds global position pos[r]
    if kind != "contiguous":
        assert np.any(np.diff(pos) < 0)
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)      # in packed (participant) order
    o, lse = oracle.sync(q, k, v, kv_pos=pos, q_pos=pos)
    inv = np.argsort(pos)                                   # packed row of global position t
    g = Hq // Hkv
    tq = torch.from_numpy(q[inv]).permute(1, 0, 2)
    tk = torch.from_numpy(np.repeat(k[inv], g, axis=1)).permute(1, 0, 2)
    tv = torch.from_numpy(np.repeat(v[inv], g, axis=1)).permute(1, 0, 2)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(1, 0, 2).numpy()
    assert np.abs(o[inv] - want).max() < 1e-12
    n = 2                                                   # one participant's rows against the global KV
    r0 = sum(lens[:n])
    rows = np.arange(r0, r0 + lens[n])
    o_n, lse_n = oracle.sync(q[rows], k, v, kv_pos=pos, q_pos=pos[rows])
    bo, bl = brute_attention(q[rows], lambda j, kvh: k[j, kvh], lambda j, kvh: v[j, kvh],
                             lambda i, h: ([j for j in range(L) if pos[j] <= pos[rows[i]]], h // g), 1 / math.sqrt(d))
    assert np.abs(o_n - bo).max() < 1e-12 and np.abs(lse_n - bl).max() < 1e-12
    assert np.abs(o_n - o[rows]).max() < 1e-13


def test_gqa_equals_mha_with_repeated_kv_heads(oracle):
    lens = [6, 5]
    L, Hq, Hkv, d = sum(lens), 6, 2, 8
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    kr, vr = np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1)
    assert np.array_equal(oracle.local(q, k, v, lens)[0], oracle.local(q, kr, vr, lens)[0])
    assert np.array_equal(oracle.sync(q, k, v)[0], oracle.sync(q, kr, vr)[0])


def test_decode_equals_last_prefill_row(oracle):
    """A decode query placed after the cache sees every cached row: it equals the last row of
    the prefill result when the cache holds the same K/V (local: last row of the segment;
    sync: last row of the global sequence)."""
    lens = [6, 6, 6]
    N, cap, Hq, Hkv, d = 3, 6, 4, 2, 8
    L = sum(lens)
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    o_loc, lse_loc = oracle.local(q, k, v, lens)
    last = np.cumsum(lens) - 1
    qd = q[last]
    o_d, lse_d = oracle.decode(qd, k.reshape(N, cap, Hkv, d), v.reshape(N, cap, Hkv, d), lens, False)
    assert np.abs(o_d - o_loc[last]).max() < 1e-13 and np.abs(lse_d - lse_loc[last]).max() < 1e-13
    # shorter kv_len than capacity: only the first rows count
    o_d2, _ = oracle.decode(qd, k.reshape(N, cap, Hkv, d), v.reshape(N, cap, Hkv, d), [6, 2, 4], False)
    o_p2, _ = oracle.sync(qd[1:2], k[6:8], v[6:8], causal=False)
    assert np.abs(o_d2[1] - o_p2[0]).max() < 1e-13
    # sync: every participant's query sees the whole global cache
    o_s, lse_s = oracle.decode(qd, k, v, [L], True)
    o_full, lse_full = oracle.sync(qd, k, v, causal=False)
    assert np.abs(o_s - o_full).max() < 1e-13 and np.abs(lse_s - lse_full).max() < 1e-13
    o_cen, _ = oracle.sync(q, k, v)
    assert np.abs(o_s[-1] - o_cen[-1]).max() < 1e-13


def test_row_subset_matches_full(oracle):
    lens = [9, 4]
    L, H, d = 13, 2, 4
    q, k, v = randn(L, H, d), randn(L, H, d), randn(L, H, d)
    rows = [0, 8, 9, 12]
    assert np.array_equal(oracle.local(q, k, v, lens, rows=rows)[0], oracle.local(q, k, v, lens)[0][rows])
    assert np.array_equal(oracle.sync(q, k, v, rows=rows)[1], oracle.sync(q, k, v)[1][rows])


def test_block_schedule_matches_printed_marginal_savings():
    """The number of sync blocks is M / H; the saving when H grows to H+1, as a fraction of the
    H=1 cost, is 1/(H(H+1)) -- values printed in the paper (golden file)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "schedule_marginal_savings.txt")
    M = 2 * 3 * 4 * 5
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        H, num, den = (int(x) for x in line.split())
        rounds = lambda h: sum(fi.is_sync_block(m, h) for m in range(1, M + 1))
        assert rounds(H) == M // H
        assert Fraction(rounds(H) - rounds(H + 1), rounds(1)) == Fraction(num, den)
    assert [sum(fi.is_sync_block(m, H) for m in range(1, 33)) for H in (1, 2, 4, 8, 32)] == [32, 16, 8, 4, 1]
    assert fi.is_sync_block(32, 32) and not fi.is_sync_block(31, 32)


def test_variable_round_schedule_reduces_to_uniform():
    """Theorem 3's setting: H_t local forwards in round t, sum H_t = M; the uniform case is H_t = H."""
    M = 32
    for H in (1, 2, 4, 8, 32):
        assert fi.sync_blocks_of_rounds([H] * (M // H)) == [m for m in range(1, M + 1) if fi.is_sync_block(m, H)]
    assert fi.sync_blocks_of_rounds([2, 6, 10, 14]) == [2, 8, 18, 32]        # intervals growing with depth
    assert sum([14, 10, 6, 2]) == M and fi.sync_blocks_of_rounds([14, 10, 6, 2])[-1] == M
    with pytest.raises(ValueError):
        fi.sync_blocks_of_rounds([4, 0, 4])



def test_participant_subset_exchange_reduces_to_local_and_to_dense_sync(oracle):
    """Adaptive aggregation (a participant mask per round): members send every row, the others none.
    One member alone sees only its own keys, i.e. its local attention; all members give the dense
    sync block; in between, a member's row sees exactly the members' keys at or before its position."""
    lens = [5, 3, 6, 4]
    L, Hq, Hkv, d = sum(lens), 4, 2, 4
    off = np.concatenate([[0], np.cumsum(lens)])
    q, k, v = randn(L, Hq, d), randn(L, Hkv, d), randn(L, Hkv, d)
    cuts = np.cumsum(lens)[:-1]
    ks, vs = np.split(k, cuts), np.split(v, cuts)
    o_loc, lse_loc = oracle.local(q, k, v, lens)
    o_den, lse_den = oracle.sync(q, k, v)
    for members in ([2], [0, 1, 2, 3], [1, 3]):
        ksel = [lens[n] if n in members else 0 for n in range(4)]
        ka, va, pos, cu, sel = oracle.aggregate_topk(ks, vs, ksel)
        want_pos = np.concatenate([np.arange(off[n], off[n + 1]) for n in members])
        assert np.array_equal(pos, np.tile(want_pos, (Hkv, 1))) and cu[-1] == len(want_pos)
        rows = want_pos.astype(np.int32)
        o, lse = oracle.sync(q[rows], ka, va, kv_pos=pos, q_pos=rows, kv_head_major=True)
        if len(members) == 1:
            assert np.allclose(o, o_loc[rows], atol=1e-12) and np.allclose(lse, lse_loc[rows], atol=1e-12)
        elif len(members) == 4:
            assert np.allclose(o, o_den, atol=1e-12) and np.allclose(lse, lse_den, atol=1e-12)
        else:
            g = Hq // Hkv
            ob, lb = brute_attention(q[rows], lambda j, kvh: k[j, kvh], lambda j, kvh: v[j, kvh],
                                     lambda i, h: ([int(j) for j in want_pos if j <= rows[i]], h // g),
                                     1.0 / math.sqrt(d))
            assert np.allclose(o, ob, atol=1e-12) and np.allclose(lse, lb, atol=1e-12)


def test_decode_over_global_cache_plus_private_suffix_is_the_merge_of_two_decodes(oracle):
    """A sync-block decode step after generation has begun: the shared global cache followed by the
    participant's own new rows.  Softmax over a disjoint union = log-sum-exp merge of the parts."""
    n, T, cap, Hq, Hkv, d = 3, 11, 4, 4, 2, 4
    kg, vg = randn(T, Hkv, d), randn(T, Hkv, d)
    ksx, vsx = randn(n, cap, Hkv, d), randn(n, cap, Hkv, d)
    q = randn(n, Hq, d)
    sfx = [4, 0, 2]
    o_g, lse_g = oracle.decode(q, kg, vg, [T], True)
    o_s, lse_s = oracle.decode(q, ksx, vsx, sfx, False)
    assert np.all(o_s[1] == 0) and np.all(np.isneginf(lse_s[1]))
    cat_k = np.concatenate([np.broadcast_to(kg, (n,) + kg.shape), ksx], axis=1)
    cat_v = np.concatenate([np.broadcast_to(vg, (n,) + vg.shape), vsx], axis=1)
    o, lse = oracle.decode(q, cat_k, cat_v, [T + s for s in sfx], False)
    om, lm = lse_merge(o_g, lse_g, o_s, lse_s)
    assert np.allclose(o, om, atol=1e-12) and np.allclose(lse, lm, atol=1e-12)


def test_input_generators_are_seeded_and_typed():
    w = fi.cfg2()
    a = fi.normal(2, fi.TENSOR_Q, 0, (4, 3), "bf16")
    b = fi.normal(2, fi.TENSOR_Q, 0, (4, 3), "bf16")
    assert np.array_equal(a, b)
    assert np.array_equal(torch.from_numpy(a).to(torch.bfloat16).float().numpy(), a)
    x = np.array([1.00390625, 1.01171875, -1.00390625, 3.0e-40], dtype=np.float32)  # ties to even
    assert np.array_equal(fi.round_to_bf16(x), torch.from_numpy(x).to(torch.bfloat16).float().numpy())
    assert w.total_tokens == 8192 and fi.cfg4().k_sel == 256
    lens = fi.cfg3().seqlens
    assert len(lens) == 8 and all(256 <= x <= 4096 for x in lens)
    rows = fi.sample_rows(3, lens, 64)
    assert rows.min() >= 0 and rows.max() < sum(lens) and 0 in rows and sum(lens) - 1 in rows
