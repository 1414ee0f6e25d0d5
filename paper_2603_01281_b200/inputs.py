"""Seeded synthetic workloads shaped like the paper's models.

This module only draws inputs; it holds none of the method's arithmetic and is
the one module shared by the CUDA-path tests and the CPU checker.  Tensors are
packed ``[total_tokens, heads, d]`` float32 numpy arrays whose values are exactly
representable in the workload's storage type (bf16 values are rounded to nearest
even here, so both sides start from identical numbers).

Recipes (seed = 260301281 + index of the configuration):
  C1  toy layer: B=1, 4 heads (MHA), d=64, L=256, fp32, rank 8, one highlighted
      span of 32 tokens, g=0.5
  C2  8B-shaped prefill layer: B=4, 32 query / 8 KV heads, d=128, L=4096, bf16,
      rank 32, 1-3 highlighted spans covering 10 % of each sequence, g=1
  C3  AdaSEKA on the 8B shape: B=2, L=8192, M=4 experts of rank 32, 10 %, g=1
  C4  long context: B=1, 28 query / 4 KV heads, d=128, L=32768, rank 64,
      8 scattered spans of 64-512 tokens (about 5 %), g=2
  C5  batched varlen small model: 64 sequences, lengths uniform in [256, 2048],
      16/16 heads, d=64, bf16, rank 16, highlight runs (runs of 1-16 tokens,
      each highlighted with p=0.15), g uniform in [0.25, 2] per sequence
  C2s70 / C2s100  C2 with one middle span of 70 % of the tokens / everything
      highlighted (the paper's own overhead run steers most of a long context)
Q, K, V are i.i.d. N(0,1); each U is the first r columns of the orthogonal factor
of a seeded d x d Gaussian (the paper's random-projection ablation input), signs
fixed so the triangular factor has a positive diagonal; singular values for the
experts are sigma_k = s_m * 0.9**k with s_m uniform in [0.5, 2].
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

BASE_SEED = 260301281


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


@dataclass
class Workload:
    name: str
    dtype: str                      # "f32" or "bf16": storage type of Q, K, V, O
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rank: int
    n_experts: int
    cu_seqlens: np.ndarray          # int32 [B+1]
    fixed_len: Optional[int]        # L when every sequence has the same length, else None
    Q: np.ndarray
    K: np.ndarray
    V: np.ndarray
    mask: np.ndarray                # uint8 [total]
    U: np.ndarray                   # float32 [M, Hkv, d, r]
    gain: np.ndarray                # float32 [B]
    sigma: Optional[np.ndarray] = None   # float32 [M, Hkv, r] (experts only)
    head_enable: Optional[np.ndarray] = None
    k_route: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.cu_seqlens) - 1

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def max_seqlen(self) -> int:
        return int(np.max(np.diff(self.cu_seqlens))) if self.batch else 0

    def attention_flops(self) -> float:
        """Causal QK^T + PV flops, 2 per multiply-add; the edit is not credited."""
        Ls = np.diff(self.cu_seqlens).astype(np.float64)
        return float(4.0 * self.head_dim * self.n_q_heads * np.sum(Ls * (Ls + 1.0) / 2.0))


def orthonormal_bank(rng: np.random.Generator, M: int, Hkv: int, d: int, r: int) -> np.ndarray:
    U = np.empty((M, Hkv, d, r), dtype=np.float32)
    for m in range(M):
        for h in range(Hkv):
            Qf, Rf = np.linalg.qr(rng.standard_normal((d, d)))
            Qf = Qf * np.sign(np.diag(Rf))[None, :]
            U[m, h] = Qf[:, :r].astype(np.float32)
    return U


def expert_sigma(rng: np.random.Generator, M: int, Hkv: int, r: int) -> np.ndarray:
    s = rng.uniform(0.5, 2.0, size=(M, Hkv, 1))
    return (s * 0.9 ** np.arange(r)[None, None, :]).astype(np.float32)


def span_mask(rng: np.random.Generator, L: int, lengths) -> np.ndarray:
    """Disjoint highlighted spans of the given lengths at seeded offsets (gaps >= 1 between spans)."""
    lengths = [int(x) for x in lengths if int(x) > 0]
    n = len(lengths)
    free = L - sum(lengths) - (n - 1)
    assert free >= 0, "spans do not fit"
    cuts = np.sort(rng.integers(0, free + 1, size=n))
    gaps = np.diff(np.concatenate([[0], cuts]))
    m = np.zeros(L, dtype=np.uint8)
    pos = 0
    for k, ln in enumerate(lengths):
        pos += int(gaps[k]) + (1 if k > 0 else 0)
        m[pos:pos + ln] = 1
        pos += ln
    return m


def split_total(rng: np.random.Generator, total: int, n: int) -> list:
    """Split ``total`` into n positive parts at seeded cut points."""
    if n <= 1 or total <= n:
        return [total]
    cuts = np.sort(rng.choice(np.arange(1, total), size=n - 1, replace=False))
    return list(np.diff(np.concatenate([[0], cuts, [total]])).astype(int))


def run_mask(rng: np.random.Generator, L: int, p: float = 0.15, max_run: int = 16) -> np.ndarray:
    """Consecutive runs of 1..max_run tokens, each run highlighted independently with probability p."""
    m = np.zeros(L, dtype=np.uint8)
    pos = 0
    while pos < L:
        ln = int(rng.integers(1, max_run + 1))
        if rng.random() < p:
            m[pos:pos + ln] = 1
        pos += ln
    return m


_RECIPES = {
    # name: (index, dtype, B, Hq, Hkv, d, L, r, M, g)
    "C1": (0, "f32", 1, 4, 4, 64, 256, 8, 1, 0.5),
    "C2": (1, "bf16", 4, 32, 8, 128, 4096, 32, 1, 1.0),
    "C3": (2, "bf16", 2, 32, 8, 128, 8192, 32, 4, 1.0),
    "C4": (3, "bf16", 1, 28, 4, 128, 32768, 64, 1, 2.0),
    "C5": (4, "bf16", 64, 16, 16, 64, None, 16, 1, None),
    "C2s70": (5, "bf16", 4, 32, 8, 128, 4096, 32, 1, 1.0),
    "C2s100": (6, "bf16", 4, 32, 8, 128, 4096, 32, 1, 1.0),
}


def make_workload(name: str, *, batch: Optional[int] = None, seqlen: Optional[int] = None,
                  min_len: int = 256, max_len: int = 2048, n_q_heads: Optional[int] = None,
                  n_kv_heads: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """Build one of the named configurations; the keyword overrides shrink it for tests."""
    idx, dtype, B, Hq, Hkv, d, L, r, M, g = _RECIPES[name]
    B = batch if batch is not None else B
    L = seqlen if (seqlen is not None and L is not None) else L
    Hq = n_q_heads if n_q_heads is not None else Hq
    Hkv = n_kv_heads if n_kv_heads is not None else Hkv
    rng = np.random.default_rng(BASE_SEED + idx + 1000 * seed_offset)

    if L is None:
        lens = rng.integers(min_len, max_len + 1, size=B)
    else:
        lens = np.full(B, L)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1])

    def draw(h):
        x = rng.standard_normal((total, h, d), dtype=np.float32)
        return round_to_bf16(x) if dtype == "bf16" else x

    Q, K, V = draw(Hq), draw(Hkv), draw(Hkv)
    U = orthonormal_bank(rng, M, Hkv, d, r)
    sigma = expert_sigma(rng, M, Hkv, r) if M > 1 else None

    mask = np.zeros(total, dtype=np.uint8)
    for b in range(B):
        Lb = int(lens[b])
        if name == "C1":
            mb = span_mask(rng, Lb, [min(32, Lb)])
        elif name in ("C2", "C3"):
            n = int(rng.integers(1, 4))
            mb = span_mask(rng, Lb, split_total(rng, int(round(0.10 * Lb)), n))
        elif name == "C4":
            ls = rng.integers(64, 513, size=8).astype(np.float64)
            ls = np.maximum(1, np.round(ls * (0.05 * Lb) / ls.sum())).astype(int)
            mb = span_mask(rng, Lb, ls)
        elif name == "C5":
            mb = run_mask(rng, Lb)
        elif name == "C2s70":
            ln = int(round(0.70 * Lb)); st = (Lb - ln) // 2
            mb = np.zeros(Lb, dtype=np.uint8); mb[st:st + ln] = 1
        elif name == "C2s100":
            mb = np.ones(Lb, dtype=np.uint8)
        else:
            raise KeyError(name)
        mask[cu[b]:cu[b + 1]] = mb

    if g is None:
        gain = rng.uniform(0.25, 2.0, size=B).astype(np.float32)
    else:
        gain = np.full(B, g, dtype=np.float32)

    return Workload(name=name, dtype=dtype, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, rank=r, n_experts=M,
                    cu_seqlens=cu, fixed_len=(int(L) if L is not None else None), Q=Q, K=K, V=V, mask=mask,
                    U=U, gain=gain, sigma=sigma, k_route=0,
                    meta={"seed": BASE_SEED + idx + 1000 * seed_offset,
                          "highlight_fraction": float(mask.mean()) if total else 0.0})


def make_custom(*, seed: int, dtype: str, lens, n_q_heads: int, n_kv_heads: int, head_dim: int, rank: int,
                n_experts: int = 1, mask_kind: str = "spans", gain=1.0, highlight: float = 0.1) -> Workload:
    """Free-form workload for edge-case tests (same distributions as the named recipes)."""
    rng = np.random.default_rng(seed)
    lens = np.asarray(lens, dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1]); d = head_dim

    def draw(h):
        x = rng.standard_normal((total, h, d), dtype=np.float32)
        return round_to_bf16(x) if dtype == "bf16" else x

    Q, K, V = draw(n_q_heads), draw(n_kv_heads), draw(n_kv_heads)
    U = orthonormal_bank(rng, n_experts, n_kv_heads, d, rank)
    sigma = expert_sigma(rng, n_experts, n_kv_heads, rank) if n_experts > 1 else None
    mask = np.zeros(total, dtype=np.uint8)
    for b, Lb in enumerate(lens):
        Lb = int(Lb)
        if Lb == 0:
            continue
        if mask_kind == "spans":
            T = min(Lb, max(1, int(round(highlight * Lb))))
            mb = span_mask(rng, Lb, split_total(rng, T, int(rng.integers(1, 4))))
        elif mask_kind == "runs":
            mb = run_mask(rng, Lb, p=highlight)
        elif mask_kind == "all":
            mb = np.ones(Lb, dtype=np.uint8)
        elif mask_kind == "none":
            mb = np.zeros(Lb, dtype=np.uint8)
        else:
            raise KeyError(mask_kind)
        mask[cu[b]:cu[b + 1]] = mb
    B = len(lens)
    gain = np.broadcast_to(np.asarray(gain, dtype=np.float32), (B,)).copy()
    fixed = int(lens[0]) if B and np.all(lens == lens[0]) else None
    return Workload(name="custom", dtype=dtype, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=d, rank=rank,
                    n_experts=n_experts, cu_seqlens=cu, fixed_len=fixed, Q=Q, K=K, V=V, mask=mask, U=U, gain=gain,
                    sigma=sigma, meta={"seed": seed})


def sample_rows(rng: np.random.Generator, L: int, mask: np.ndarray, n: int, tile: int = 128) -> np.ndarray:
    """Query rows for sampled parity: first/last, tile edges, rows just after each span, plus random rows."""
    if L <= n:
        return np.arange(L, dtype=np.int32)
    must = {0, L - 1}
    for t in range(tile, L, tile):
        must.update((t - 1, t))
    m = np.asarray(mask[:L]) != 0
    ends = np.flatnonzero(m[:-1] & ~m[1:]) + 1
    starts = np.flatnonzero(~m[:-1] & m[1:]) + 1
    for e in list(ends[:8]) + list(starts[:8]):
        must.update((int(e), min(L - 1, int(e) + 1)))
    must = sorted(x for x in must if 0 <= x < L)
    if len(must) > n:
        keep = {0, L - 1}
        rest = [x for x in must if x not in keep]
        pick = rng.choice(len(rest), size=n - 2, replace=False)
        must = sorted(keep | {rest[i] for i in pick})
    extra = n - len(must)
    if extra > 0:
        pool = np.setdiff1d(np.arange(L), np.asarray(must))
        must = sorted(set(must) | set(rng.choice(pool, size=extra, replace=False).tolist()))
    return np.asarray(must, dtype=np.int32)


def contrastive_embeddings(*, seed: int, n: int, slots: int, head_dim: int, rank: int = 8, dtype: str = "bf16"):
    """Synthetic stand-in for the key embeddings of the paper's contrastive prompts (Section 3.1): for each of
    `slots` (layer, KV head) pairs, n neutral keys with a decaying per-dimension spread (0.98**j), and positive /
    negative keys in which a planted `rank`-dimensional relevance subspace is amplified by a_s / attenuated by
    a_s / 2 (a_s uniform in [0.3, 1.5]; every fourth slot has a_s = 0, i.e. a head that does not react), plus
    N(0, 0.1) noise.  Also a Bernoulli(0.3) set of "answer tokens".  Returns float32 arrays h, h_pos, h_neg
    [n, slots, d] (rounded to the storage type), answer_tokens uint8 [n], the planted bases [slots, d, rank] and
    the strengths a_s.  Draws only; none of the learning arithmetic lives here."""
    rng = np.random.default_rng(BASE_SEED + 1000 + seed)
    d = head_dim
    decay = (0.98 ** np.arange(d)).astype(np.float64)
    h = np.empty((n, slots, d), dtype=np.float32); hp = np.empty_like(h); hn = np.empty_like(h)
    bases = np.empty((slots, d, rank), dtype=np.float64)
    strength = rng.uniform(0.3, 1.5, size=slots)
    strength[3::4] = 0.0
    for s in range(slots):
        q, _ = np.linalg.qr(rng.standard_normal((d, rank)))
        bases[s] = q
        z = rng.standard_normal((n, d)) * decay
        lift = (z @ q) @ q.T
        h[:, s] = z
        hp[:, s] = z + strength[s] * lift + 0.1 * rng.standard_normal((n, d))
        hn[:, s] = z - 0.5 * strength[s] * lift + 0.1 * rng.standard_normal((n, d))
    if dtype == "bf16":
        h, hp, hn = round_to_bf16(h), round_to_bf16(hp), round_to_bf16(hn)
    answer = (rng.random(n) < 0.3).astype(np.uint8)
    return h, hp, hn, answer, bases, strength
