"""Shared plumbing of the GPU parity tests: moves seeded numpy inputs to the device, calls the
CUDA path through the C-ABI binding and returns numpy float64 results."""
from __future__ import annotations

import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2}     # max-abs bounds: fp32 inputs / bf16 inputs with O(1) outputs
LSE_TOL = {"f32": 1e-4, "bf16": 1e-3}  # log-sum-exp (fp32 output): fp32 inputs / bf16 inputs


def fa():
    import paper_2511_02647_b200 as m
    return m


def dev(x: np.ndarray, dtype: str):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.cuda()


def host(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def make_shape(n, hq, hkv, d, dtype, causal=True, scale=0.0):
    m = fa()
    return m.Shape(n, hq, hkv, d, m.BF16 if dtype == "bf16" else m.F32, int(causal), scale)


class Runner:
    """One library context sized for the given limits."""

    def __init__(self, n, hq, hkv, d, dtype, max_tokens, max_kv=None, causal=True, scale=0.0):
        self.m = fa()
        self.dtype = dtype
        self.shape = make_shape(n, hq, hkv, d, dtype, causal, scale)
        self.ctx = self.m.Context(self.shape, max_tokens, max_kv if max_kv is not None else max_tokens)
        self.n, self.hq, self.hkv, self.d = n, hq, hkv, d

    def poll(self):
        return self.ctx.poll()

    def local(self, q, k, v, seqlens, want_lse=True):
        cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int64)
        qd, kd, vd = dev(q, self.dtype), dev(k, self.dtype), dev(v, self.dtype)
        o = torch.full_like(qd, float("nan"))
        lse = torch.full((q.shape[0], self.hq), float("nan"), device="cuda") if want_lse else None
        self.m.fedattn_local(self.ctx, self.shape, qd, kd, vd, cu, o, lse)
        assert self.poll() == 0
        return host(o), (host(lse) if want_lse else None)

    def aggregate(self, mode, k_parts, v_parts, k_sel=None, sel_idx_in=None):
        """Returns dict of device tensors: k_agg, v_agg, kv_pos, cu_kv, sel_idx."""
        m = self.m
        seqlens = [int(x.shape[0]) for x in k_parts]
        kd = [dev(x, self.dtype) for x in k_parts]
        vd = [dev(x, self.dtype) for x in v_parts]
        td = self.shape.torch_dtype
        if mode == m.AGG_CONCAT:
            L = sum(seqlens)
            out = dict(k_agg=torch.zeros((L, self.hkv, self.d), dtype=td, device="cuda"),
                       v_agg=torch.zeros((L, self.hkv, self.d), dtype=td, device="cuda"),
                       kv_pos=torch.full((L,), -1, dtype=torch.int32, device="cuda"),
                       cu_kv=torch.full((self.n + 1,), -1, dtype=torch.int32, device="cuda"), sel_idx=None)
            m.fedattn_aggregate_kv(self.ctx, self.shape, mode, kd, vd, seqlens, None, None, out["k_agg"],
                                   out["v_agg"], out["kv_pos"], out["cu_kv"], None)
        elif mode == m.AGG_TOPK_TOKEN:
            T = int(sum(k_sel))
            out = dict(k_agg=torch.zeros((T, self.hkv, self.d), dtype=td, device="cuda"),
                       v_agg=torch.zeros((T, self.hkv, self.d), dtype=td, device="cuda"),
                       kv_pos=torch.full((T,), -1, dtype=torch.int32, device="cuda"),
                       cu_kv=torch.full((self.n + 1,), -1, dtype=torch.int32, device="cuda"),
                       sel_idx=torch.full((T,), -1, dtype=torch.int32, device="cuda"))
            m.fedattn_aggregate_kv(self.ctx, self.shape, mode, kd, vd, seqlens, list(k_sel), None, out["k_agg"],
                                   out["v_agg"], out["kv_pos"], out["cu_kv"], out["sel_idx"])
        else:
            T = int(sum(k_sel))
            out = dict(k_agg=torch.zeros((self.hkv, T, self.d), dtype=td, device="cuda"),
                       v_agg=torch.zeros((self.hkv, T, self.d), dtype=td, device="cuda"),
                       kv_pos=torch.full((self.hkv, T), -1, dtype=torch.int32, device="cuda"),
                       cu_kv=torch.full((self.n + 1,), -1, dtype=torch.int32, device="cuda"),
                       sel_idx=torch.full((self.hkv, T), -1, dtype=torch.int32, device="cuda"))
            sel_in = None if sel_idx_in is None else torch.from_numpy(
                np.ascontiguousarray(sel_idx_in, dtype=np.int32)).cuda()
            m.fedattn_aggregate_kv(self.ctx, self.shape, mode, kd, vd, seqlens, list(k_sel), sel_in, out["k_agg"],
                                   out["v_agg"], out["kv_pos"], out["cu_kv"], out["sel_idx"])
        out["status"] = self.poll()
        return out

    def sync(self, q, k_agg, v_agg, kv_pos=None, q_pos=None, head_major=False, want_lse=True):
        """k_agg/v_agg/kv_pos: device tensors (from aggregate) or numpy arrays."""
        qd = dev(q, self.dtype)
        if isinstance(k_agg, np.ndarray):
            k_agg, v_agg = dev(k_agg, self.dtype), dev(v_agg, self.dtype)
        if isinstance(kv_pos, np.ndarray):
            kv_pos = torch.from_numpy(np.ascontiguousarray(kv_pos, dtype=np.int32)).cuda()
        if isinstance(q_pos, np.ndarray):
            q_pos = torch.from_numpy(np.ascontiguousarray(q_pos, dtype=np.int32)).cuda()
        T = k_agg.shape[1] if head_major else k_agg.shape[0]
        o = torch.full_like(qd, float("nan"))
        lse = torch.full((q.shape[0], self.hq), float("nan"), device="cuda") if want_lse else None
        self.m.fedattn_sync(self.ctx, self.shape, qd, q_pos, k_agg, v_agg, kv_pos, T, head_major, o, lse)
        assert self.poll() == 0
        return host(o), (host(lse) if want_lse else None)

    def sync_exchange(self, q, k, v, seqlens, agg):
        """Sync block with sparse KV exchange: local + remote-only sync + merge.  agg: dict from
        aggregate() (head-major sparse KV).  Returns (o, lse) as numpy float64."""
        m = self.m
        cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int64)
        qd, kd, vd = dev(q, self.dtype), dev(k, self.dtype), dev(v, self.dtype)
        L = q.shape[0]
        o_a = torch.full_like(qd, float("nan")); o_b = torch.full_like(qd, float("nan"))
        lse_a = torch.full((L, self.hq), float("nan"), device="cuda"); lse_b = torch.full_like(lse_a, float("nan"))
        o = torch.full_like(qd, float("nan")); lse = torch.full_like(lse_a, float("nan"))
        T = agg["k_agg"].shape[1]
        m.fedattn_local(self.ctx, self.shape, qd, kd, vd, cu, o_a, lse_a)
        m.fedattn_sync_remote(self.ctx, self.shape, qd, cu, agg["k_agg"], agg["v_agg"], agg["kv_pos"], T, True, o_b, lse_b)
        m.fedattn_merge(self.ctx, self.shape, L, o_a, lse_a, o_b, lse_b, o, lse)
        assert self.poll() == 0
        return host(o), host(lse)

    def merge(self, o_a, lse_a, o_b, lse_b):
        """LSE merge of two partial attention results over disjoint key sets (numpy in, numpy out)."""
        oa, ob = dev(o_a.astype(np.float32), self.dtype), dev(o_b.astype(np.float32), self.dtype)
        la = torch.from_numpy(np.ascontiguousarray(lse_a, dtype=np.float32)).cuda()
        lb = torch.from_numpy(np.ascontiguousarray(lse_b, dtype=np.float32)).cuda()
        o = torch.full_like(oa, float("nan")); lse = torch.full_like(la, float("nan"))
        self.m.fedattn_merge(self.ctx, self.shape, int(o_a.shape[0]), oa, la, ob, lb, o, lse)
        assert self.poll() == 0
        return host(o), host(lse)

    def decode(self, q, k_cache, v_cache, kv_len, sync_mode, max_kv_len=None):
        m = self.m
        qd, kd, vd = dev(q, self.dtype), dev(k_cache, self.dtype), dev(v_cache, self.dtype)
        lens = torch.tensor([int(x) for x in kv_len], dtype=torch.int32, device="cuda")
        stride = 0 if sync_mode else int(np.prod(k_cache.shape[1:]))
        o = torch.full_like(qd, float("nan"))
        lse = torch.full((q.shape[0], self.hq), float("nan"), device="cuda")
        mx = int(max(kv_len)) if max_kv_len is None else max_kv_len
        m.fedattn_decode(self.ctx, self.shape, m.DECODE_SYNC if sync_mode else m.DECODE_LOCAL, qd, kd, vd, stride,
                         lens, mx, o, lse)
        assert self.poll() == 0
        return host(o), host(lse)


def check_close(got, want, tol, what=""):
    got, want = np.asarray(got), np.asarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    fin = np.isfinite(want)
    assert np.array_equal(np.isfinite(got), fin), what + ": finite pattern differs"
    assert np.array_equal(got[~fin], want[~fin]) or not (~fin).any(), what
    err = np.abs(got[fin] - want[fin]).max() if fin.any() else 0.0
    assert err <= tol, "%s: max-abs error %.3e > %.1e" % (what, err, tol)
    return err
