"""Seeded synthetic inputs shaped like the paper's pre-ranking workload.

This module only draws numbers and lays them out; it holds none of the method's arithmetic and loads no
native code.  It feeds the CUDA library and the test oracle with the very same host arrays.

Storage convention: a "storage array" is numpy float32 (dtype "f32") or numpy uint16 holding bf16 bit
patterns (dtype "bf16"), already rounded once here so that both sides start from identical values.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Optional, Sequence, Tuple

import numpy as np

BLK_ATT, BLK_CROSS, BLK_BEA, BLK_LSH_DIN, BLK_SIMTIER = 1, 2, 4, 8, 16
BUCKET_MOD, BUCKET_HASH = 0, 1
NORM_NONE, NORM_MEAN = 0, 1
MASTER_SEED = 20251112


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(a: np.ndarray, dtype: str) -> np.ndarray:
    """float array -> storage array of the workload's type."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a if dtype == "f32" else to_bf16_bits(a)


def as_f32(a: np.ndarray, dtype: str) -> np.ndarray:
    return a if dtype == "f32" else bf16_bits_to_f32(a)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the five benchmark shapes (or a scaled-down copy of one for fast parity tests)."""
    name: str
    dtype: str                      # "f32" | "bf16"
    R: int                          # requests
    N: int                          # candidates per request (upper bound when mixed)
    M: int                          # rows of the item table
    d: int                          # width of item / user vectors
    L: int                          # behaviour-sequence length
    F: int                          # cross fields
    B: int                          # buckets per field
    dc: int                         # width of one cross embedding
    hidden: Tuple[int, ...]         # hidden widths of the scoring MLP (the output is 1 wide)
    sigma: float                    # std of the normal embeddings
    bucket_mode: int = BUCKET_HASH
    id_dist: str = "zipf"           # "uniform" | "zipf"
    zipf_s: float = 1.1
    overlap: float = 0.0            # share of each request's ids taken from one pool common to all requests
    mini_batch: int = 0             # candidates per mini-batch (0: the request is one batch)
    mixed_sizes: Optional[Tuple[int, int]] = None   # request sizes uniform in [lo, hi]
    blocks: int = BLK_ATT | BLK_CROSS
    n_bridge: int = 8
    n_tiers: int = 8
    lsh_din_norm: int = NORM_MEAN
    simtier_norm: int = NORM_MEAN
    emit_sigmoid: int = 0
    dU: int = 0                     # width of the raw user embeddings (0: same as d)
    n_cross_tables: int = 0         # distinct cross tables generated and cycled over requests (0: one per request)
    n_categories: int = 0           # item categories; > 0: the interaction blocks see the candidate's category's sub-sequence

    @property
    def raw_dU(self) -> int:
        return self.dU or self.d

    @property
    def lsh_bits(self) -> int:
        return self.d

    def input_width(self) -> int:
        w = 2 * self.d
        if self.blocks & BLK_ATT:
            w += self.d
        if self.blocks & BLK_CROSS:
            w += self.F * self.dc
        if self.blocks & BLK_BEA:
            w += self.d
        if self.blocks & BLK_LSH_DIN:
            w += self.d
        if self.blocks & BLK_SIMTIER:
            w += self.n_tiers
        return w

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five shapes of the benchmark definition.
C1 = Workload("c1_tiny_fp32", "f32", R=1, N=1000, M=100_000, d=64, L=50, F=8, B=16, dc=16, hidden=(256, 128),
              sigma=0.1, bucket_mode=BUCKET_MOD, id_dist="uniform", emit_sigmoid=1,
              lsh_din_norm=NORM_NONE, simtier_norm=NORM_NONE)
C2 = Workload("c2_paper_shaped", "bf16", R=1, N=10_000, M=1_000_000, d=128, L=200, F=16, B=1024, dc=32,
              hidden=(512, 256), sigma=0.05, mini_batch=1000)
C3 = Workload("c3_concurrent", "bf16", R=64, N=10_000, M=10_000_000, d=128, L=1000, F=16, B=1024, dc=32,
              hidden=(512, 256), sigma=0.05, overlap=0.3)
C4 = Workload("c4_long_sequence", "bf16", R=16, N=10_000, M=1_000_000, d=128, L=10_000, F=16, B=1024, dc=32,
              hidden=(512, 256), sigma=0.05)
C5 = Workload("c5_wide", "bf16", R=256, N=4000, M=5_000_000, d=256, L=500, F=64, B=4096, dc=32,
              hidden=(1024, 512, 256), sigma=0.05, n_cross_tables=16)
C5_MIXED = C5.with_(name="c5_wide_mixed", N=10_000, mixed_sizes=(1000, 10_000))
# the long-sequence shape with the LSH blocks (eqs. 6-9) in place of, and beside, the dense target attention
C4_LSH = C4.with_(name="c4_long_sequence_lsh", blocks=BLK_CROSS | BLK_LSH_DIN | BLK_SIMTIER)
C4_BOTH = C4.with_(name="c4_long_sequence_att_lsh", blocks=BLK_ATT | BLK_CROSS | BLK_LSH_DIN | BLK_SIMTIER)
C4_DIN = C4.with_(name="c4_long_sequence_lsh_din", blocks=BLK_CROSS | BLK_LSH_DIN)
# the long-term sequence of Sections 3.3 / 4.2 (length ~10^5): LSH blocks over the whole sequence, and attention + LSH blocks
# over the candidate's category's sub-sequence (100 categories, SIM-hard)
LONG_LSH = C4.with_(name="long_1e5_lsh", R=4, L=100_000, blocks=BLK_CROSS | BLK_LSH_DIN | BLK_SIMTIER)
LONG_SIM = C4.with_(name="long_1e5_sim", R=4, L=100_000, blocks=BLK_ATT | BLK_CROSS | BLK_LSH_DIN | BLK_SIMTIER, n_categories=100)
CONFIGS = {w.name: w for w in (C1, C2, C3, C4, C5, C5_MIXED, C4_LSH, C4_BOTH, C4_DIN, LONG_LSH, LONG_SIM)}
SHORT = {"c1": C1, "c2": C2, "c3": C3, "c4": C4, "c5": C5, "c5a": C5, "c5b": C5_MIXED, "c4_lsh": C4_LSH, "c4_both": C4_BOTH,
         "c4_din": C4_DIN, "long_lsh": LONG_LSH, "long_sim": LONG_SIM}


def _seed(*keys) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([MASTER_SEED] + [int(k) for k in keys]))


def _tag(name: str) -> int:
    h = 0
    for ch in name.encode():
        h = (h * 131 + ch) % (2**31 - 1)
    return h


def normal_rows(rows: int, cols: int, sigma: float, dtype: str, *keys, threads: int = 8) -> np.ndarray:
    """[rows x cols] N(0, sigma) storage array; drawn in fixed row chunks so that the result does not
    depend on the number of threads."""
    out = np.empty((rows, cols), dtype=np.float32 if dtype == "f32" else np.uint16)
    chunk = 1 << 16
    starts = list(range(0, rows, chunk))

    def fill(i):
        lo = starts[i]
        hi = min(rows, lo + chunk)
        g = _seed(*keys, i)
        a = g.standard_normal((hi - lo, cols), dtype=np.float32) * np.float32(sigma)
        out[lo:hi] = store(a, dtype)

    if len(starts) == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(len(starts))))
    return out


def glorot_uniform(rows: int, cols: int, dtype: str, *keys) -> np.ndarray:
    """[rows x cols] weight, U(-a, a) with a = sqrt(6 / (rows + cols))."""
    a = np.sqrt(6.0 / (rows + cols))
    g = _seed(*keys)
    return store(g.uniform(-a, a, size=(rows, cols)).astype(np.float32), dtype)


def make_weights(wl: Workload, zero_bias: bool = True) -> dict:
    """Scoring MLP (input = full concatenated vector) and user-side network weights."""
    t = _tag(wl.name)
    widths = [wl.input_width()] + list(wl.hidden)
    W, b = [], []
    for k in range(len(wl.hidden)):
        W.append(glorot_uniform(widths[k + 1], widths[k], wl.dtype, t, 100 + k))
        if zero_bias:
            b.append(np.zeros(widths[k + 1], dtype=np.float32))
        else:
            b.append((_seed(t, 150 + k).standard_normal(widths[k + 1]) * 0.05).astype(np.float32))
    w_out = glorot_uniform(1, widths[-1], wl.dtype, t, 190).reshape(-1)
    b_out = np.zeros(1, dtype=np.float32) if zero_bias else np.full(1, 0.125, dtype=np.float32)
    d, dU = wl.d, wl.raw_dU
    user = {
        "W_profile": glorot_uniform(d, dU, wl.dtype, t, 200),
        "W_seq": glorot_uniform(d, dU, wl.dtype, t, 201),
        "W_a": glorot_uniform(d, d, wl.dtype, t, 202),
        "W_b": glorot_uniform(d, d, wl.dtype, t, 203),
        "b_a": np.zeros(d, dtype=np.float32) if zero_bias else (_seed(t, 204).standard_normal(d) * 0.05).astype(np.float32),
        "b_b": np.zeros(d, dtype=np.float32) if zero_bias else (_seed(t, 205).standard_normal(d) * 0.05).astype(np.float32),
    }
    if wl.blocks & BLK_BEA:   # user side of Algorithm 1: bridges B ~ N(0, 1) (a softmax that is not flat), W_f Glorot
        user["bridges"] = normal_rows(wl.n_bridge, d, 1.0, wl.dtype, t, 414)
        user["W_f"] = glorot_uniform(d, d, wl.dtype, t, 206)
    return {"mlp": {"W": W, "b": b, "w_out": w_out, "b_out": b_out}, "user": user}


def _signatures(rows: int, nbytes: int, *keys, protos: Optional[np.ndarray] = None) -> np.ndarray:
    """Packed binary signatures with structure: every row is a prototype with a row-specific share of
    its bits flipped, so that agreement counts between rows spread over a wide range."""
    g = _seed(*keys)
    nbits = nbytes * 8
    if protos is None:
        protos = g.integers(0, 2, size=(16, nbits), dtype=np.uint8)
    which = g.integers(0, protos.shape[0], size=rows)
    flip_p = g.uniform(0.0, 0.5, size=(rows, 1))
    bits = protos[which] ^ (g.random((rows, nbits)) < flip_p).astype(np.uint8)
    return np.packbits(bits, axis=1, bitorder="big")


def signature_prototypes(wl: Workload) -> np.ndarray:
    return _seed(_tag(wl.name), 300).integers(0, 2, size=(16, wl.lsh_bits), dtype=np.uint8)


def make_item_table(wl: Workload, rows: Optional[int] = None) -> dict:
    """E [M x d] (+ the BEA weight rows and the LSH signatures when those blocks are on)."""
    t = _tag(wl.name)
    M = rows or wl.M
    tab = {"E": normal_rows(M, wl.d, wl.sigma, wl.dtype, t, 1)}
    if wl.blocks & BLK_BEA:
        g = _seed(t, 2)
        tab["bea_w"] = store(g.dirichlet(np.ones(wl.n_bridge), size=M).astype(np.float32), wl.dtype)
    if wl.blocks & (BLK_LSH_DIN | BLK_SIMTIER):
        tab["sig"] = _signatures(M, wl.lsh_bits // 8, t, 3, protos=signature_prototypes(wl))
    return tab


def make_item_side(wl: Workload, n: int, dI: Optional[int] = None, hI: Optional[int] = None, d_mm: Optional[int] = None) -> dict:
    """Inputs and weights of the item side of the nearline pipeline for n items: raw features I_raw [n x dI] (dI = 4 d by
    default: the paper reports item-side compression of more than 3x), id embeddings I_id [n x d], multi-modal
    embeddings M_mm [n x d_mm]; tower weights (Glorot uniform, small biases), bridges B [n_bridge x d] ~ N(0, 1) (so that
    the softmax over bridges is not flat), W_hash [lsh_bits x d_mm] ~ N(0, 1) in storage type."""
    t = _tag(wl.name)
    dI, hI, d_mm = dI or 4 * wl.d, hI or 2 * wl.d, d_mm or wl.d
    out = {
        "I_raw": normal_rows(n, dI, wl.sigma, wl.dtype, t, 400),
        "I_id": normal_rows(n, wl.d, 1.0, wl.dtype, t, 401),
        "M_mm": normal_rows(n, d_mm, 1.0, wl.dtype, t, 402),
        "W_i0": glorot_uniform(hI, dI, wl.dtype, t, 410),
        "W_i1": glorot_uniform(wl.d, hI, wl.dtype, t, 411),
        "b_i0": (_seed(t, 412).standard_normal(hI) * 0.05).astype(np.float32),
        "b_i1": (_seed(t, 413).standard_normal(wl.d) * 0.05).astype(np.float32),
        "bridges": normal_rows(max(wl.n_bridge, 1), wl.d, 1.0, wl.dtype, t, 414),
        "W_hash": normal_rows(max(wl.lsh_bits, 8), d_mm, 1.0, wl.dtype, t, 415),
    }
    return out


class IdSampler:
    """Candidate ids: distinct within a request; uniform, or Zipf(s) ranks mapped through a fixed random
    permutation of the rows; an optional pool shared by all requests gives cross-request overlap."""

    def __init__(self, wl: Workload, M: Optional[int] = None):
        self.wl = wl
        self.M = M or wl.M
        t = _tag(wl.name)
        if wl.id_dist == "zipf":
            w = np.arange(1, self.M + 1, dtype=np.float64) ** (-wl.zipf_s)
            self.cdf = np.cumsum(w)
            self.cdf /= self.cdf[-1]
            self.perm = _seed(t, 10).permutation(self.M).astype(np.int32)
        self.pool = None
        if wl.overlap > 0:
            self.pool = self._draw(_seed(t, 11), int(round(wl.overlap * wl.N)), None)

    def _raw(self, g, k):
        if self.wl.id_dist == "uniform":
            return g.integers(0, self.M, size=k).astype(np.int32)
        ranks = np.searchsorted(self.cdf, g.random(k), side="left")
        return self.perm[np.minimum(ranks, self.M - 1)]

    def _draw(self, g, k, exclude):
        seen = set() if exclude is None else set(int(x) for x in exclude)
        out = []
        while len(out) < k:
            for v in self._raw(g, max(64, 2 * (k - len(out)))):
                v = int(v)
                if v not in seen:
                    seen.add(v)
                    out.append(v)
                    if len(out) == k:
                        break
        return np.asarray(out, dtype=np.int32)

    def request_ids(self, r: int, n: Optional[int] = None) -> np.ndarray:
        wl = self.wl
        g = _seed(_tag(wl.name), 12, r)
        if n is None:
            n = wl.N if wl.mixed_sizes is None else int(g.integers(wl.mixed_sizes[0], wl.mixed_sizes[1] + 1))
        if self.pool is None:
            return self._draw(g, n, None)
        k = min(len(self.pool), int(round(wl.overlap * n)))
        own = self._draw(g, n - k, self.pool[:k])
        ids = np.concatenate([self.pool[:k], own])
        return ids[g.permutation(n)].astype(np.int32)


def make_request(wl: Workload, r: int, L: Optional[int] = None) -> dict:
    """User-side inputs of request r.

    "profile" [dU] and "seq" [L x dU] are the raw embeddings for the user-side network; "u" [d] and "S"
    [L x d] are a combined user vector and a projected sequence for callers that supply them directly.
    "T" [F x B x dc], "V" [n x d], "sig_seq" [L x d'/8] as enabled; "seq_cat" [L] the category of every sequence item
    when the workload has categories."""
    t = _tag(wl.name)
    L = L or wl.L
    dU = wl.raw_dU
    rq = {
        "profile": normal_rows(1, dU, wl.sigma, wl.dtype, t, 20, r).reshape(-1),
        "seq": normal_rows(L, dU, wl.sigma, wl.dtype, t, 21, r),
        "u": normal_rows(1, wl.d, wl.sigma, wl.dtype, t, 22, r).reshape(-1),
        "S": normal_rows(L, wl.d, wl.sigma, wl.dtype, t, 23, r),
    }
    if wl.blocks & BLK_CROSS:
        tr = r % wl.n_cross_tables if wl.n_cross_tables else r
        rq["T"] = normal_rows(wl.F * wl.B, wl.dc, wl.sigma, wl.dtype, t, 24, tr).reshape(wl.F, wl.B, wl.dc)
    if wl.blocks & BLK_BEA:
        rq["V"] = normal_rows(wl.n_bridge, wl.d, wl.sigma, wl.dtype, t, 25, r)
    if wl.blocks & (BLK_LSH_DIN | BLK_SIMTIER):
        rq["sig_seq"] = _signatures(L, wl.lsh_bits // 8, t, 26, r, protos=signature_prototypes(wl))
    if wl.n_categories > 0:
        # a user's behaviours are skewed towards a few categories: weights 1 / (rank + 1) over a per-request order
        g = _seed(t, 27, r)
        w = 1.0 / (1.0 + g.permutation(wl.n_categories))
        rq["seq_cat"] = g.choice(wl.n_categories, size=L, p=w / w.sum()).astype(np.int32)
    return rq
