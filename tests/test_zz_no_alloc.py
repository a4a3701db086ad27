"""fedattn_decode_noalloc: the decode entry point for callers that cannot allocate device memory
(no context, no workspace; its split-KV scratch is a fixed array inside the library).  It must give
what fedattn_decode gives, and what the fp64 oracle gives.  Two calls in a row with different inputs also show that whatever the
previous call left in the shared scratch does not leak into the next result.  This file sorts
last so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

import fedattn_inputs as fi
from helpers import TOL, fa, host

pytestmark = pytest.mark.gpu


def _run_pair(m, shape, ctx, mode, q, k, v, stride, lens, max_len, want):
    """fedattn_decode_noalloc against fedattn_decode, and against the fp64 oracle's result `want`."""
    o_ref = torch.full_like(q, float("nan")); o_new = torch.full_like(q, float("nan"))
    lse_ref = torch.full(q.shape[:2], float("nan"), device="cuda"); lse_new = torch.full_like(lse_ref, float("nan"))
    m.fedattn_decode(ctx, shape, mode, q, k, v, stride, lens, max_len, o_ref, lse_ref)
    assert ctx.poll() == 0
    m.fedattn_decode_noalloc(shape, mode, q, k, v, stride, lens, max_len, o_new, lse_new)
    torch.cuda.synchronize()
    err = np.abs(host(o_new) - host(o_ref)).max()
    assert np.isfinite(host(o_new)).all() and err <= TOL["bf16"], err
    assert np.abs(host(lse_new) - host(lse_ref)).max() <= 1e-3
    assert np.abs(host(o_new) - want[0]).max() <= TOL["bf16"]
    assert np.abs(host(lse_new) - want[1]).max() <= 1e-3


def test_noalloc_decode_matches_decode_twice_in_a_row(oracle):
    m = fa()
    n, cap, hq, hkv, d = 8, 1024, 32, 8, 128
    w = fi.Workload("noalloc", 21, (cap,) * n, hq, hkv, d, "bf16")
    shape = m.Shape(n, hq, hkv, d, m.BF16)
    ctx = m.Context(shape, n * cap, n * cap)
    bf = torch.bfloat16
    for call in range(2):                       # second call: new K/V/q, shorter ragged lengths
        _, kn, vn = w.qkv(block=call)
        qn = w.decode_q(call)
        q = torch.from_numpy(qn).to(bf).cuda()
        k = torch.from_numpy(kn).to(bf).cuda(); v = torch.from_numpy(vn).to(bf).cuda()
        lens_l = [cap] * n if call == 0 else [cap - 37 * i for i in range(n)]
        lens = torch.tensor(lens_l, dtype=torch.int32, device="cuda")
        want = oracle.decode(qn, kn.reshape(n, cap, hkv, d), vn.reshape(n, cap, hkv, d), lens_l, False)
        _run_pair(m, shape, ctx, m.DECODE_LOCAL, q, k, v, cap * hkv * d, lens, cap, want)
        t_len = n * cap - 100 * call
        tot = torch.tensor([t_len], dtype=torch.int32, device="cuda")
        want = oracle.decode(qn, kn, vn, [t_len], True)
        _run_pair(m, shape, ctx, m.DECODE_SYNC, q, k, v, 0, tot, n * cap, want)


def test_noalloc_decode_rejects_what_its_scratch_cannot_hold():
    m = fa()
    z = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    lens = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(m.FedAttnError) as e:    # 16 * 32 = 512 output rows > 256
        m.fedattn_decode_noalloc(m.Shape(16, 32, 8, 128, m.BF16), m.DECODE_SYNC, z, z, z, 0, lens, 64, z)
    assert e.value.code == 3
    with pytest.raises(m.FedAttnError) as e:    # fp32 has no kernel behind this entry point
        m.fedattn_decode_noalloc(m.Shape(2, 4, 2, 128, m.F32), m.DECODE_SYNC, z, z, z, 0, lens, 64, z)
    assert e.value.code == 2
