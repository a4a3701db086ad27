"""Stream order of calls that start early (programmatic dependent launch): chains of aggregation and
decode calls over shared buffers, issued back to back without a host synchronisation, must give what
the same calls give one at a time.  Expected values come from the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

import fedattn_inputs as fi
from helpers import LSE_TOL, TOL, check_close, dev, fa, host, make_shape

pytestmark = pytest.mark.gpu

N, L, KSEL, HQ, HKV, D = 8, 1024, 512, 8, 2, 128


def _case(seed):
    w = fi.Workload("order", seed, (L,) * N, HQ, HKV, D, "bf16")
    _, k, v = w.qkv()
    lens = [L] * N
    kp, vp = np.split(k, np.cumsum(lens)[:-1]), np.split(v, np.cumsum(lens)[:-1])
    return w.decode_q(0), kp, vp


class _Chain:
    """Two input sets A and B aggregated (token-level top-k) into ONE set of output buffers, each
    aggregation followed by a sync decode that reads those buffers."""

    def __init__(self, oracle):
        m = fa()
        self.m = m
        self.shape = make_shape(N, HQ, HKV, D, "bf16")
        self.ctx = m.Context(self.shape, N * L, N * L)
        T = N * KSEL
        self.T = T
        bf = torch.bfloat16
        self.k_agg = torch.zeros((T, HKV, D), dtype=bf, device="cuda")
        self.v_agg = torch.zeros_like(self.k_agg)
        self.kv_pos = torch.zeros((T,), dtype=torch.int32, device="cuda")
        self.cu_kv = torch.zeros((N + 1,), dtype=torch.int32, device="cuda")
        self.sel = torch.zeros((T,), dtype=torch.int32, device="cuda")
        self.lens = torch.tensor([T], dtype=torch.int32, device="cuda")
        self.sets, self.want = [], []
        for seed in (71, 72):
            q, kp, vp = _case(seed)
            ka, va, _, _, _ = oracle.aggregate_topk_token(kp, vp, [KSEL] * N)
            self.want.append(oracle.decode(q, ka, va, [T], True))
            self.sets.append((dev(q, "bf16"), [dev(x, "bf16") for x in kp], [dev(x, "bf16") for x in vp]))

    def aggregate(self, i, stream=None):
        _, kd, vd = self.sets[i]
        self.m.fedattn_aggregate_kv(self.ctx, self.shape, self.m.AGG_TOPK_TOKEN, kd, vd, [L] * N, [KSEL] * N, None,
                                    self.k_agg, self.v_agg, self.kv_pos, self.cu_kv, self.sel, stream=stream)

    def decode(self, i, o, lse, stream=None):
        self.m.fedattn_decode(self.ctx, self.shape, self.m.DECODE_SYNC, self.sets[i][0], self.k_agg, self.v_agg, 0,
                              self.lens, self.T, o, lse, stream=stream)

    def check(self, i, o, lse, what):
        check_close(host(o), self.want[i][0], TOL["bf16"], what + " o")
        check_close(host(lse), self.want[i][1], LSE_TOL["bf16"], what + " lse")


def test_aggregation_into_buffers_a_running_decode_still_reads(oracle):
    """aggregate(A) -> decode -> aggregate(B) -> decode -> ... over one set of output buffers: the second
    aggregation must not overwrite rows the first decode has yet to read, the decode must not read rows
    the aggregation has yet to write."""
    c = _Chain(oracle)
    reps = 24
    o = torch.full((reps, 2, N, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((reps, 2, N, HQ), float("nan"), device="cuda")
    for r in range(reps):
        for i in (0, 1):
            c.aggregate(i)
            c.decode(i, o[r, i], lse[r, i])
    torch.cuda.synchronize()
    assert c.ctx.poll() == 0
    for r in range(reps):
        for i in (0, 1):
            c.check(i, o[r, i], lse[r, i], "rep %d set %d" % (r, i))


def test_repeated_aggregation_into_the_same_buffers_then_one_reader(oracle):
    """aggregate(A), aggregate(B), aggregate(A), ... back to back into the same buffers (each may write
    as soon as the one before it is over), then one decode: it sees the last one's rows."""
    c = _Chain(oracle)
    o = torch.full((4, N, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((4, N, HQ), float("nan"), device="cuda")
    for t, n_calls in enumerate((1, 2, 7, 16)):
        for j in range(n_calls):
            c.aggregate(j & 1)
        c.decode((n_calls - 1) & 1, o[t], lse[t])
    torch.cuda.synchronize()
    assert c.ctx.poll() == 0
    for t, n_calls in enumerate((1, 2, 7, 16)):
        c.check((n_calls - 1) & 1, o[t], lse[t], "%d aggregations" % n_calls)


def test_chain_on_two_streams_with_events_and_in_a_replayed_graph(oracle):
    """The same chain with the context moving between two streams (ordered by events), and captured once
    into a CUDA graph that is replayed: every replay orders its calls like the first."""
    c = _Chain(oracle)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    o = torch.full((6, 2, N, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((6, 2, N, HQ), float("nan"), device="cuda")
    torch.cuda.synchronize()
    prev = None
    for r in range(6):
        for i in (0, 1):
            s = (s1, s2)[(r + i) & 1]
            if prev is not None:
                s.wait_event(prev)
            c.aggregate(i, stream=s.cuda_stream)
            c.decode(i, o[r, i], lse[r, i], stream=s.cuda_stream)
            prev = torch.cuda.Event()
            prev.record(s)
    torch.cuda.synchronize()
    assert c.ctx.poll() == 0
    for r in range(6):
        for i in (0, 1):
            c.check(i, o[r, i], lse[r, i], "two streams rep %d set %d" % (r, i))

    og = torch.full((2, N, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lg = torch.full((2, N, HQ), float("nan"), device="cuda")
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        g.capture_begin()
        for i in (0, 1, 0, 1):
            c.aggregate(i, stream=side.cuda_stream)
            c.decode(i, og[i], lg[i], stream=side.cuda_stream)
        g.capture_end()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(5):
        og.fill_(float("nan"))
        g.replay()
        c.aggregate(0)                       # an eager call between replays, into the same buffers
    torch.cuda.synchronize()
    assert c.ctx.poll() == 0
    for i in (0, 1):
        c.check(i, og[i], lg[i], "graph replay set %d" % i)


def test_indexed_gather_right_behind_the_selection_that_writes_its_indices(oracle):
    """top-k per KV head (writes the kept indices) -> indexed gather with exactly those indices, back to
    back and alternating between two input sets: the gather starts early but must not read indices the
    selection has yet to write; its rows are the selection's own rows, bit for bit."""
    m = fa()
    shape = make_shape(N, HQ, HKV, D, "bf16")
    ctx = m.Context(shape, N * L, N * L)
    T = N * KSEL
    bf = torch.bfloat16
    k1 = torch.zeros((HKV, T, D), dtype=bf, device="cuda"); v1 = torch.zeros_like(k1)
    k2 = torch.zeros_like(k1); v2 = torch.zeros_like(k1)
    pos1 = torch.zeros((HKV, T), dtype=torch.int32, device="cuda"); pos2 = torch.zeros_like(pos1)
    sel = torch.zeros_like(pos1); cu1 = torch.zeros((N + 1,), dtype=torch.int32, device="cuda"); cu2 = torch.zeros_like(cu1)
    sets, want = [], []
    for seed in (81, 82):
        _, kp, vp = _case(seed)
        ka, va, pa, _, _ = oracle.aggregate_topk(kp, vp, [KSEL] * N)
        want.append((ka, va, pa))
        sets.append(([dev(x, "bf16") for x in kp], [dev(x, "bf16") for x in vp]))
    reps = 12
    got_k = torch.zeros((reps, 2) + tuple(k2.shape), dtype=bf, device="cuda")
    got_v = torch.zeros_like(got_k)
    got_p = torch.zeros((reps, 2) + tuple(pos2.shape), dtype=torch.int32, device="cuda")
    for r in range(reps):
        for i in (0, 1):
            kd, vd = sets[i]
            m.fedattn_aggregate_kv(ctx, shape, m.AGG_TOPK_KNORM, kd, vd, [L] * N, [KSEL] * N, None, k1, v1, pos1, cu1, sel)
            m.fedattn_aggregate_kv(ctx, shape, m.AGG_INDEXED, kd, vd, [L] * N, [KSEL] * N, sel, k2, v2, pos2, cu2, None)
            got_k[r, i].copy_(k2); got_v[r, i].copy_(v2); got_p[r, i].copy_(pos2)
    torch.cuda.synchronize()
    assert ctx.poll() == 0
    for r in range(reps):
        for i in (0, 1):
            assert np.array_equal(host(got_k[r, i]), want[i][0]), (r, i)
            assert np.array_equal(host(got_v[r, i]), want[i][1]), (r, i)
            assert np.array_equal(got_p[r, i].cpu().numpy(), want[i][2]), (r, i)


# ---------------------------------------------------------------------------------------------
# An invariance, not a parity: a seeded random sequence of calls over shared buffers gives, bit for
# bit, what the same sequence gives with a host synchronisation after every call.  (Each call's parity
# with the oracle is tested elsewhere; this draws the orders in which buffers are written, read and
# written again by calls that start early.)
# ---------------------------------------------------------------------------------------------
def _fa():
    return fa()


def _random_sequence(seed, sync_every, n_ops=60):
    fa = _fa()
    bf = torch.bfloat16
    N, L, KS, HQ, HKV, D = 4, 512, 256, 8, 2, 128
    T, KS2 = N * KS, KS // 2
    T2 = N * KS2
    shape = fa.Shape(N, HQ, HKV, D, fa.BF16)
    torch.manual_seed(1234)
    ctx = fa.Context(shape, N * L, N * L)
    g = torch.Generator(device='cuda'); g.manual_seed(77)
    parts = [[(torch.randn(L, HKV, D, device='cuda', generator=g).to(bf), torch.randn(L, HKV, D, device='cuda', generator=g).to(bf)) for _ in range(N)] for _ in range(2)]
    q = torch.randn(N, HQ, D, device='cuda', generator=g).to(bf)
    qp = torch.randn(T, HQ, D, device='cuda', generator=g).to(bf)
    tok_k = torch.zeros(T, HKV, D, dtype=bf, device='cuda'); tok_v = torch.zeros_like(tok_k)
    tok_pos = torch.zeros(T, dtype=torch.int32, device='cuda'); tok_cu = torch.zeros(N + 1, dtype=torch.int32, device='cuda'); tok_sel = torch.zeros(T, dtype=torch.int32, device='cuda')
    t2_k = torch.zeros(T2, HKV, D, dtype=bf, device='cuda'); t2_v = torch.zeros_like(t2_k)
    t2_pos = torch.zeros(T2, dtype=torch.int32, device='cuda'); t2_cu = torch.zeros(N + 1, dtype=torch.int32, device='cuda'); t2_sel = torch.zeros(T2, dtype=torch.int32, device='cuda')
    sp_k = torch.zeros(HKV, T, D, dtype=bf, device='cuda'); sp_v = torch.zeros_like(sp_k)
    sp_pos = torch.zeros(HKV, T, dtype=torch.int32, device='cuda'); sp_cu = torch.zeros(N + 1, dtype=torch.int32, device='cuda'); sp_sel = torch.zeros(HKV, T, dtype=torch.int32, device='cuda')
    ix_k = torch.zeros_like(sp_k); ix_v = torch.zeros_like(sp_k); ix_pos = torch.zeros_like(sp_pos); ix_cu = torch.zeros_like(sp_cu)
    o_dec = torch.zeros(N, HQ, D, dtype=bf, device='cuda'); lse_dec = torch.zeros(N, HQ, device='cuda')
    o_pre = torch.zeros(T, HQ, D, dtype=bf, device='cuda')
    lensT = torch.tensor([T], dtype=torch.int32, device='cuda'); lensT2 = torch.tensor([T2], dtype=torch.int32, device='cuda')
    have_sel = False
    rng = np.random.default_rng(seed)
    log = []
    def snap(*ts): log.append([t.clone() for t in ts])
    for op in range(n_ops):
        c = int(rng.integers(0, 8)); i = int(rng.integers(0, 2))
        kd = [p[0] for p in parts[i]]; vd = [p[1] for p in parts[i]]
        if c == 0:
            fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_TOPK_TOKEN, kd, vd, [L] * N, [KS] * N, None, tok_k, tok_v, tok_pos, tok_cu, tok_sel)
        elif c == 1:
            fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_TOPK_KNORM, kd, vd, [L] * N, [KS] * N, None, sp_k, sp_v, sp_pos, sp_cu, sp_sel); have_sel = True
        elif c == 2 and have_sel:
            fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_INDEXED, kd, vd, [L] * N, [KS] * N, sp_sel, ix_k, ix_v, ix_pos, ix_cu, None); snap(ix_k, ix_pos)
        elif c == 3:
            fa.fedattn_decode(ctx, shape, fa.DECODE_SYNC, q, tok_k, tok_v, 0, lensT, T, o_dec, lse_dec); snap(o_dec, lse_dec)
        elif c == 4:   # second-level selection: the token-level aggregate, cut in N parts, is the input
            k2 = [tok_k[n * KS:(n + 1) * KS] for n in range(N)]; v2 = [tok_v[n * KS:(n + 1) * KS] for n in range(N)]
            fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_TOPK_TOKEN, k2, v2, [KS] * N, [KS2] * N, None, t2_k, t2_v, t2_pos, t2_cu, t2_sel)
        elif c == 5:
            fa.fedattn_decode(ctx, shape, fa.DECODE_SYNC, q, t2_k, t2_v, 0, lensT2, T2, o_dec, lse_dec); snap(o_dec, lse_dec)
        elif c == 6:   # prefill over the sparse aggregate (reads what 1 wrote), then its output feeds nothing
            fa.fedattn_sync(ctx, shape, qp, None, sp_k, sp_v, sp_pos if have_sel else None, T, True, o_pre); snap(o_pre)
        elif c == 7:   # local decode over the raw parts of set i laid out as caches: uses tok buffers as caches of N x KS rows
            lens = torch.full((N,), KS, dtype=torch.int32, device='cuda')
            fa.fedattn_decode(ctx, shape, fa.DECODE_LOCAL, q, tok_k, tok_v, KS * HKV * D, lens, KS, o_dec, lse_dec); snap(o_dec, lse_dec)
        if sync_every: torch.cuda.synchronize()
    torch.cuda.synchronize()
    st = ctx.poll()
    return log, st


@pytest.mark.parametrize("seed", range(8))
def test_seeded_random_call_sequences_match_their_synchronised_run(seed):
    a, status_a = _random_sequence(seed, True)
    b, status_b = _random_sequence(seed, False)
    assert status_a == 0 and status_b == 0 and len(a) == len(b) and len(a) > 0
    for n, (x, y) in enumerate(zip(a, b)):
        assert all(torch.equal(p, r) for p, r in zip(x, y)), "snapshot %d of %d differs" % (n, len(a))
