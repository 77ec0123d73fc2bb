"""ctypes front end of the CPU oracle (oracle/aif_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the bench's cpu_baseline and
reference legs.  It knows nothing of the CUDA library and shares no code with it.

Arrays in "storage type" are numpy float32 (dtype "f32") or numpy uint16 holding bf16 bit patterns
(dtype "bf16"); the C side widens them exactly to double.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
from typing import Optional, Sequence

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
BUCKET_MOD, BUCKET_HASH = 0, 1
BLK_ATT, BLK_CROSS, BLK_BEA, BLK_LSH_DIN, BLK_SIMTIER = 1, 2, 4, 8, 16
NORM_NONE, NORM_MEAN = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.orc_mix64.restype = C.c_uint64
        _lib.orc_mix64.argtypes = [C.c_uint64, C.c_uint64]
        _lib.orc_bucket.restype = C.c_int64
        _lib.orc_bucket.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
        _lib.orc_category.restype = C.c_int64
        _lib.orc_category.argtypes = [C.c_int64, C.c_int, C.c_int]
        _lib.orc_mlp.restype = C.c_double
        _lib.orc_num_threads.restype = C.c_int
    return _lib


class _Cfg(C.Structure):
    _fields_ = [
        ("dtype", C.c_int32), ("M", C.c_int64), ("d", C.c_int32), ("F", C.c_int32), ("B", C.c_int32),
        ("dc", C.c_int32), ("n_hidden", C.c_int32), ("hidden", C.c_int32 * 4), ("bucket_mode", C.c_int32),
        ("blocks", C.c_int32), ("n_bridge", C.c_int32), ("lsh_bits", C.c_int32), ("n_tiers", C.c_int32),
        ("lsh_din_norm", C.c_int32), ("simtier_norm", C.c_int32), ("emit_sigmoid", C.c_int32), ("n_categories", C.c_int32),
    ]


class _Mlp(C.Structure):
    _fields_ = [("W", C.c_void_p * 4), ("b", C.c_void_p * 4), ("w_out", C.c_void_p), ("b_out", C.c_void_p)]


class _UserW(C.Structure):
    _fields_ = [("W_profile", C.c_void_p), ("W_seq", C.c_void_p), ("W_a", C.c_void_p), ("b_a", C.c_void_p),
                ("W_b", C.c_void_p), ("b_b", C.c_void_p)]


class _Req(C.Structure):
    _fields_ = [("E", C.c_void_p), ("bea_w", C.c_void_p), ("sig", C.c_void_p), ("u", C.c_void_p),
                ("S", C.c_void_p), ("l", C.c_int32), ("T", C.c_void_p), ("V", C.c_void_p),
                ("sig_seq", C.c_void_p), ("seq_cat", C.c_void_p)]


@dataclasses.dataclass
class OracleConfig:
    dtype: int
    M: int
    d: int
    F: int = 0
    B: int = 1
    dc: int = 0
    hidden: Sequence[int] = (256, 128)
    bucket_mode: int = BUCKET_MOD
    blocks: int = BLK_ATT | BLK_CROSS
    n_bridge: int = 8
    lsh_bits: int = 0
    n_tiers: int = 8
    lsh_din_norm: int = NORM_NONE
    simtier_norm: int = NORM_NONE
    emit_sigmoid: int = 0
    n_categories: int = 0

    def c(self) -> _Cfg:
        h = list(self.hidden) + [0] * (4 - len(self.hidden))
        return _Cfg(self.dtype, self.M, self.d, self.F, self.B, self.dc, len(self.hidden), (C.c_int32 * 4)(*h),
                    self.bucket_mode, self.blocks, self.n_bridge, self.lsh_bits, self.n_tiers,
                    self.lsh_din_norm, self.simtier_norm, self.emit_sigmoid, self.n_categories)

    def input_width(self) -> int:
        cfg = self.c()
        return int(lib().orc_input_width(C.byref(cfg)))


def _store(a: Optional[np.ndarray], dtype: int) -> Optional[np.ndarray]:
    """Checks that an array is in the storage type and contiguous."""
    if a is None:
        return None
    want = np.float32 if dtype == F32 else np.uint16
    if a.dtype != want:
        raise TypeError(f"storage array must be {want}, got {a.dtype}")
    return np.ascontiguousarray(a)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def widen(a: np.ndarray, dtype: int) -> np.ndarray:
    """Storage array -> float64 (exact)."""
    if dtype == F32:
        return a.astype(np.float64)
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ------------------------------------------------------------------------------------------------
# element functions
# ------------------------------------------------------------------------------------------------
def mix64(id_: int, field: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(id_ & (2**64 - 1)), C.c_uint64(field)))


def bucket(id_: int, field: int, B: int, mode: int) -> int:
    return int(lib().orc_bucket(id_, field, B, mode))


def category(id_: int, n_categories: int, mode: int) -> int:
    return int(lib().orc_category(id_, n_categories, mode))


CATEGORY_FIELD = 3239


def pack_bits(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.zeros(bits.size // 8, dtype=np.uint8)
    lib().orc_pack_bits(_p(bits), C.c_int(bits.size), _p(out))
    return out


def popcount_lut(v: int) -> int:
    return int(lib().orc_popcount_lut(C.c_int(v)))


def lsh_matches(a: np.ndarray, b: np.ndarray, via_lut: bool = True) -> int:
    a = np.ascontiguousarray(a, dtype=np.uint8)
    b = np.ascontiguousarray(b, dtype=np.uint8)
    return int(lib().orc_lsh_matches(_p(a), _p(b), C.c_int(a.size), C.c_int(1 if via_lut else 0)))


def lsh_hash_bits(m, W_hash) -> np.ndarray:
    m = _f64(m)
    W_hash = _f64(W_hash)
    dbits, d = W_hash.shape
    bits = np.zeros(dbits, dtype=np.uint8)
    lib().orc_lsh_hash_bits(_p(m), _p(W_hash), C.c_int(d), C.c_int(dbits), _p(bits))
    return bits


def lsh_similarity(sig_items: np.ndarray, sig_seq: np.ndarray, dbits: int) -> np.ndarray:
    a = np.ascontiguousarray(sig_items, dtype=np.uint8)
    s = np.ascontiguousarray(sig_seq, dtype=np.uint8)
    b, l = a.shape[0], s.shape[0]
    sim = np.zeros((b, l), dtype=np.float64)
    lib().orc_lsh_similarity(_p(a), C.c_int(b), _p(s), C.c_int(l), C.c_int(dbits), _p(sim))
    return sim


def lsh_din(sim_row, S, norm: int = NORM_NONE) -> np.ndarray:
    sim_row, S = _f64(sim_row), _f64(S)
    l, d = S.shape
    out = np.zeros(d)
    lib().orc_lsh_din(_p(sim_row), _p(S), C.c_int(l), C.c_int(d), C.c_int(norm), _p(out))
    return out


def tier_of(matches: int, dbits: int, n_tiers: int) -> int:
    return int(lib().orc_tier_of(C.c_int(matches), C.c_int(dbits), C.c_int(n_tiers)))


def simtier(matches, dbits: int, n_tiers: int, norm: int = NORM_NONE) -> np.ndarray:
    m = np.ascontiguousarray(matches, dtype=np.int32)
    out = np.zeros(n_tiers)
    lib().orc_simtier(_p(m), C.c_int(m.size), C.c_int(dbits), C.c_int(n_tiers), C.c_int(norm), _p(out))
    return out


def attention(q, S) -> np.ndarray:
    q, S = _f64(q), _f64(S)
    l, d = S.shape
    out = np.zeros(d)
    lib().orc_attention(_p(q), _p(S), C.c_int(l), C.c_int(d), _p(out))
    return out


def bea(w_hat, V) -> np.ndarray:
    w_hat, V = _f64(w_hat), _f64(V)
    n, dp = V.shape
    out = np.zeros(dp)
    lib().orc_bea(_p(w_hat), _p(V), C.c_int(n), C.c_int(dp), _p(out))
    return out


def item_nearline(dtype: int, I_raw=None, W0=None, b0=None, W1=None, b1=None, I_id=None, bridges=None, M_mm=None,
                  W_hash=None) -> dict:
    """Item side of the nearline pipeline for n items (Section 3.2 eq. 4, Algorithm 1 step 3, Section 4.2 eq. 5).
    Arrays in storage type (biases float32).  Returns the parts whose inputs were given: "I_hat" [n x d] float64,
    "w_hat" [n x n_bridge] float64, "sig" [n x dbits/8] uint8."""
    out = {}
    n = next(a.shape[0] for a in (I_raw, I_id, M_mm) if a is not None)
    I_hat = w_hat = sig = None
    dI = hI = d = nb = d_mm = dbits = 0
    if I_raw is not None:
        I_raw, W0, W1 = _store(I_raw, dtype), _store(W0, dtype), _store(W1, dtype)
        b0, b1 = np.ascontiguousarray(b0, dtype=np.float32), np.ascontiguousarray(b1, dtype=np.float32)
        (hI, dI), d = W0.shape, W1.shape[0]
        assert I_raw.shape == (n, dI) and W1.shape == (d, hI) and b0.shape == (hI,) and b1.shape == (d,)
        I_hat = np.zeros((n, d))
    if I_id is not None:
        I_id, bridges = _store(I_id, dtype), _store(bridges, dtype)
        nb, d = bridges.shape
        assert I_id.shape == (n, d) and nb <= 64
        w_hat = np.zeros((n, nb))
    if M_mm is not None:
        M_mm, W_hash = _store(M_mm, dtype), _store(W_hash, dtype)
        dbits, d_mm = W_hash.shape
        assert M_mm.shape == (n, d_mm) and dbits % 8 == 0 and dbits <= 1024
        sig = np.zeros((n, dbits // 8), dtype=np.uint8)
    lib().orc_item_nearline(C.c_int(dtype), C.c_int64(n), C.c_int(dI), C.c_int(hI), C.c_int(d), _p(I_raw), _p(W0), _p(b0),
                            _p(W1), _p(b1), _p(I_hat), C.c_int(nb), _p(I_id), _p(bridges), _p(w_hat), C.c_int(d_mm),
                            C.c_int(dbits), _p(M_mm), _p(W_hash), _p(sig))
    if I_hat is not None:
        out["I_hat"] = I_hat
    if w_hat is not None:
        out["w_hat"] = w_hat
    if sig is not None:
        out["sig"] = sig
    return out


def bea_user(dtype: int, bridges: np.ndarray, U: np.ndarray, W_f: np.ndarray):
    """Algorithm 1 steps 1-2: returns (V [n x d], W [n x m]) in float64; inputs in storage type."""
    bridges, U, W_f = _store(bridges, dtype), _store(U, dtype), _store(W_f, dtype)
    n, d = bridges.shape
    m = U.shape[0]
    assert U.shape == (m, d) and W_f.shape == (d, d)
    V, W = np.zeros((n, d)), np.zeros((n, m))
    lib().orc_bea_user(C.c_int(dtype), C.c_int(n), C.c_int(m), C.c_int(d), _p(bridges), _p(U), _p(W_f), _p(V), _p(W))
    return V, W


def lsh_projections(dtype: int, M_mm: np.ndarray, W_hash: np.ndarray) -> np.ndarray:
    """The projections M W_hash^T [n x dbits] whose signs eq. 5 keeps."""
    M_mm, W_hash = _store(M_mm, dtype), _store(W_hash, dtype)
    n, d_mm = M_mm.shape
    dbits = W_hash.shape[0]
    proj = np.zeros((n, dbits))
    lib().orc_lsh_projections(C.c_int(dtype), C.c_int64(n), C.c_int(d_mm), C.c_int(dbits), _p(M_mm), _p(W_hash), _p(proj))
    return proj


def table_refresh(table: np.ndarray, ids: Optional[np.ndarray], rows: np.ndarray) -> int:
    """In-place write of `rows` into `table` (2-D, same row width); returns the number of bad ids."""
    assert table.flags.c_contiguous and rows.flags.c_contiguous and table.dtype == rows.dtype
    row_bytes = table.strides[0]
    assert rows.strides[0] == row_bytes
    if ids is not None:
        ids = np.ascontiguousarray(ids, dtype=np.int32)
    fn = lib().orc_table_refresh
    fn.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]
    return int(fn(table.ctypes.data, table.shape[0], row_bytes, None if ids is None else ids.ctypes.data,
                  rows.shape[0], rows.ctypes.data))


# ------------------------------------------------------------------------------------------------
# whole-path functions
# ------------------------------------------------------------------------------------------------
class Oracle:
    """Holds the configuration and the weights; scores candidates one by one in fp64."""

    def __init__(self, cfg: OracleConfig, mlp: dict, user: Optional[dict] = None):
        self.cfg = cfg
        dt = cfg.dtype
        self._keep = []
        m = _Mlp()
        for k in range(len(cfg.hidden)):
            W = _store(mlp["W"][k], dt)
            b = np.ascontiguousarray(mlp["b"][k], dtype=np.float32)
            self._keep += [W, b]
            m.W[k] = W.ctypes.data
            m.b[k] = b.ctypes.data
        w_out = _store(mlp["w_out"], dt)
        b_out = np.ascontiguousarray(mlp["b_out"], dtype=np.float32).reshape(1)
        self._keep += [w_out, b_out]
        m.w_out = w_out.ctypes.data
        m.b_out = b_out.ctypes.data
        self._mlp = m
        self._user = None
        if user is not None:
            uw = _UserW()
            for name in ("W_profile", "W_seq", "W_a", "W_b"):
                a = _store(user[name], dt)
                self._keep.append(a)
                setattr(uw, name, a.ctypes.data)
            for name in ("b_a", "b_b"):
                a = np.ascontiguousarray(user[name], dtype=np.float32)
                self._keep.append(a)
                setattr(uw, name, a.ctypes.data)
            self._user = uw
            self._dU = user["W_seq"].shape[1]

    def user_state(self, profile: np.ndarray, seq: np.ndarray):
        """eqs. 1-3 from raw profile [dU] / seq [l x dU] (storage type) -> (u [d], S [l x d]) in fp64."""
        assert self._user is not None
        cfg = self.cfg.c()
        profile = _store(profile, self.cfg.dtype)
        seq = _store(seq, self.cfg.dtype)
        l = seq.shape[0]
        u = np.zeros(self.cfg.d)
        S = np.zeros((l, self.cfg.d))
        lib().orc_user_state(C.byref(cfg), C.byref(self._user), C.c_int(self._dU), _p(profile), _p(seq),
                             C.c_int(l), _p(u), _p(S))
        return u, S

    def _request(self, table: dict, request: dict):
        dt = self.cfg.dtype
        keep = []
        rq = _Req()
        E = _store(table["E"], dt)
        keep.append(E)
        rq.E = E.ctypes.data
        for name, src, conv in (("bea_w", table, lambda a: _store(a, dt)),
                                ("sig", table, lambda a: np.ascontiguousarray(a, dtype=np.uint8)),
                                ("T", request, lambda a: _store(a, dt)),
                                ("V", request, lambda a: _store(a, dt)),
                                ("sig_seq", request, lambda a: np.ascontiguousarray(a, dtype=np.uint8)),
                                ("seq_cat", request, lambda a: np.ascontiguousarray(a, dtype=np.int32))):
            a = src.get(name)
            if a is not None:
                a = conv(a)
                keep.append(a)
                setattr(rq, name, a.ctypes.data)
        u, S = _f64(request["u"]), _f64(request["S"])
        keep += [u, S]
        rq.u, rq.S, rq.l = u.ctypes.data, S.ctypes.data, S.shape[0]
        return rq, keep

    def score(self, table: dict, request: dict, ids, return_inputs: bool = False):
        """Logits (or probabilities when emit_sigmoid) of the candidates `ids` of one request.

        table: E [M x d] (+ bea_w [M x n], sig [M x d'/8]); request: u [d], S [l x d] (float64, or any
        array convertible to it exactly), T [F x B x dc], V [n x d], sig_seq [l x d'/8], seq_cat [l] (int32, needed
        when the configuration has categories)."""
        cfg = self.cfg.c()
        rq, keep = self._request(table, request)
        if self.cfg.n_categories > 0:
            assert request.get("seq_cat") is not None and len(request["seq_cat"]) == rq.l
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        out = np.zeros(ids.size)
        x = np.zeros((ids.size, self.cfg.input_width())) if return_inputs else None
        bad = lib().orc_score(C.byref(cfg), C.byref(self._mlp), C.byref(rq), _p(ids), C.c_int(ids.size), _p(out),
                              _p(x))
        self.last_bad = int(bad)
        del keep
        return (out, x) if return_inputs else out

    def mlp(self, x) -> float:
        cfg = self.cfg.c()
        x = _f64(x)
        return float(lib().orc_mlp(C.byref(cfg), C.byref(self._mlp), _p(x)))


def num_threads() -> int:
    return int(lib().orc_num_threads())
