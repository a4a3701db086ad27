"""Seeded synthetic inputs for the FedAttn attention hot path.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds no arithmetic of the method itself: it only draws random
tensors, rounds them to the storage type, draws segment lengths and lists the
workload shapes.  Neither the oracle nor the CUDA package is imported here.

Every tensor is a function of ``(seed, tensor_id, block)`` only, so any block of
a multi-block schedule can be regenerated on its own.

Workloads (shape structure only; the paper's prompts, dataset and model weights
are not available, so i.i.d. Gaussian tensors of the same shapes stand in):

* ``cfg1``  N=2 x 128 tokens, 4 heads, d=64, fp32.
* ``cfg2``  N=4 x 2048 tokens, 32 q-heads / 8 kv-heads, d=128, bf16.
* ``cfg3``  N=8, lengths uniform on [256, 4096], 32/8 heads, d=128, bf16,
  32 blocks with fresh Q/K/V per block.
* ``cfg4``  N=16 x 1024 tokens, 32/8, d=128, bf16, top 256 keys per KV head.
* ``cfg5``  decode: N=8 caches of 4096 tokens, 32/8, d=128, bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_LEN, TENSOR_MISC = 0, 1, 2, 3, 4


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32
    holding exactly representable bf16 values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def _rng(seed: int, tensor_id: int, block: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tensor_id), int(block)])


def normal(seed: int, tensor_id: int, block: int, shape, dtype: str,
           gain: float = 1.0) -> np.ndarray:
    """i.i.d. N(0, gain^2) tensor as float32, rounded to ``dtype`` ("f32"|"bf16")."""
    x = _rng(seed, tensor_id, block).standard_normal(size=shape, dtype=np.float32)
    if gain != 1.0:
        x = (x * np.float32(gain)).astype(np.float32)
    if dtype == "bf16":
        x = round_to_bf16(x)
    elif dtype != "f32":
        raise ValueError(dtype)
    return x


def uniform_lengths(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    """n integer lengths uniform on [lo, hi] (inclusive)."""
    return _rng(seed, TENSOR_LEN, 0).integers(lo, hi + 1, size=n).astype(np.int32)


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    seqlens: Tuple[int, ...]          # L_n per participant
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                        # "f32" | "bf16"
    gain: float = 1.0                 # std-dev of the Gaussian elements
    n_blocks: int = 1                 # cfg3: 32 attention calls
    k_sel: Optional[int] = None       # cfg4: keys kept per participant and KV head
    decode_steps: int = 0             # cfg5
    sync_interval: int = 1            # H for cfg5
    note: str = ""

    @property
    def n_participants(self) -> int:
        return len(self.seqlens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    def qkv(self, block: int = 0):
        """Packed Q [L,Hq,d], K [L,Hkv,d], V [L,Hkv,d] as float32 arrays whose values
        are exactly representable in ``self.dtype``."""
        L, d = self.total_tokens, self.head_dim
        q = normal(self.seed, TENSOR_Q, block, (L, self.n_q_heads, d), self.dtype, self.gain)
        k = normal(self.seed, TENSOR_K, block, (L, self.n_kv_heads, d), self.dtype, self.gain)
        v = normal(self.seed, TENSOR_V, block, (L, self.n_kv_heads, d), self.dtype, self.gain)
        return q, k, v

    def decode_q(self, step: int) -> np.ndarray:
        """One new query token per participant: [N, Hq, d]."""
        return normal(self.seed, TENSOR_MISC, step,
                      (self.n_participants, self.n_q_heads, self.head_dim),
                      self.dtype, self.gain)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def cfg1() -> Workload:
    return Workload("cfg1_fp32_2x128", 1, (128, 128), 4, 4, 64, "f32")


def cfg2() -> Workload:
    return Workload("cfg2_bf16_llama8b_4x2048", 2, (2048,) * 4, 32, 8, 128, "bf16",
                    note="elements N(0,1); softmax scale 1/sqrt(128) gives N(0,1) logits")


def cfg2_prescaled() -> Workload:
    """Literal alternative reading of the config: elements already divided by sqrt(128)."""
    return replace(cfg2(), name="cfg2_prescaled", gain=float(1.0 / np.sqrt(128.0)))


def cfg3() -> Workload:
    lens = tuple(int(x) for x in uniform_lengths(3, 8, 256, 4096))
    return Workload("cfg3_hetero_8xU256_4096", 3, lens, 32, 8, 128, "bf16", n_blocks=32)


def cfg4() -> Workload:
    return Workload("cfg4_sparse_16x1024_top256", 4, (1024,) * 16, 32, 8, 128, "bf16",
                    k_sel=256)


def cfg5() -> Workload:
    return Workload("cfg5_decode_8x4096", 5, (4096,) * 8, 32, 8, 128, "bf16",
                    decode_steps=256, sync_interval=4)


ALL = {"cfg1": cfg1, "cfg2": cfg2, "cfg3": cfg3, "cfg4": cfg4, "cfg5": cfg5}


def is_sync_block(m: int, H: int) -> bool:
    """Block m (1-based) of a schedule with sync interval H is a sync block when it is
    the H-th of its round."""
    return m % H == 0


def sync_blocks_of_rounds(local_forwards) -> List[int]:
    """Sync blocks (1-based) of a schedule given as the number of local forwards H_t of every
    communication round t: round t ends with a sync block, so the sync blocks are the running sums
    H_0, H_0 + H_1, ...  A constant H_t = H gives the uniform schedule `m mod H == 0`."""
    blocks, m = [], 0
    for h in local_forwards:
        h = int(h)
        if h <= 0:
            raise ValueError("every round needs at least one block")
        m += h
        blocks.append(m)
    return blocks


def random_subset(seed: int, participant: int, head: int, length: int, k: int) -> np.ndarray:
    """k distinct local token indices of a participant of ``length`` tokens, drawn uniformly without
    replacement from ``(seed, participant, head)`` and returned ascending: the random selector of a
    sparse KV exchange.  The draw is an input of the method, not part of it."""
    if not 0 <= k <= length:
        raise ValueError("need 0 <= k <= length")
    rng = np.random.default_rng([int(seed), TENSOR_MISC, 991, int(participant), int(head)])
    return np.sort(rng.choice(int(length), size=int(k), replace=False)).astype(np.int32)


def random_selection(seed: int, seqlens, k_sel, n_kv_heads: int) -> np.ndarray:
    """Per-head random selection for every participant in the layout the indexed aggregation
    takes: int32 [Hkv, sum k_sel], participant n's block at the prefix sum of k_sel, ascending."""
    rows = [np.concatenate([random_subset(seed, n, h, int(ln), int(k)) for n, (ln, k) in enumerate(zip(seqlens, k_sel))]
                           + [np.zeros(0, np.int32)]) for h in range(n_kv_heads)]
    return np.stack(rows).astype(np.int32)


def index_sets(seed: int, seqlens, kind: str) -> List[np.ndarray]:
    """A partition of the global positions 0..L-1 into one ascending index set per participant
    (participant n gets seqlens[n] positions).  kind = "contiguous": consecutive segments in
    participant order; "interleaved": global position t goes to the participants in round-robin
    order, skipping those that are full; "random": a seeded random assignment."""
    seqlens = [int(x) for x in seqlens]
    L = int(sum(seqlens))
    if kind == "contiguous":
        owner = np.repeat(np.arange(len(seqlens)), seqlens)
    elif kind == "interleaved":
        left = list(seqlens)
        owner = np.empty(L, dtype=np.int64)
        n = 0
        for t in range(L):
            while left[n % len(seqlens)] == 0:
                n += 1
            owner[t] = n % len(seqlens)
            left[n % len(seqlens)] -= 1
            n += 1
    elif kind == "random":
        owner = np.repeat(np.arange(len(seqlens)), seqlens)
        _rng(seed, TENSOR_MISC, 4242).shuffle(owner)
    else:
        raise ValueError(kind)
    return [np.nonzero(owner == n)[0].astype(np.int32) for n in range(len(seqlens))]


def sample_rows(seed: int, seqlens, n_random: int, tile: int = 128) -> np.ndarray:
    """Row subset for sampled parity at full size: every row within +-1 of a segment
    start/end or of a multiple of ``tile`` (both in packed and in segment-relative
    coordinates), plus ``n_random`` seeded random rows.  Sorted, unique."""
    seqlens = [int(x) for x in seqlens]
    L = int(sum(seqlens))
    rows = set()
    off = 0
    for ln in seqlens:
        for b in (off, off + ln - 1):
            for dlt in (-1, 0, 1):
                rows.add(b + dlt)
        for t in range(0, ln, tile):
            for dlt in (-1, 0, 1):
                rows.add(off + t + dlt)
        off += ln
    for t in range(0, L, tile):
        for dlt in (-1, 0, 1):
            rows.add(t + dlt)
    rnd = _rng(seed, TENSOR_MISC, 7777).integers(0, L, size=n_random)
    rows.update(int(r) for r in rnd)
    return np.array(sorted(r for r in rows if 0 <= r < L), dtype=np.int64)
