"""Thin ctypes binding of libaif.so: the same names as include/aif.h, argument marshalling only.

Every step of the scoring path runs inside the CUDA library.  There is no CPU fallback: if the library has not
been built, or no CUDA device is present, loading or creating a context raises.
PyTorch is used for device memory (torch tensors own every buffer handed to the library) and for streams.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaif.so")

OK = 0
ERR_ARG, ERR_SHAPE, ERR_OOM, ERR_CUDA, ERR_VERSION, ERR_NOT_READY, ERR_BAD_ID, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6, -7, -8
STATUS_BAD_ID, STATUS_TIMEOUT = 1, 2
F32, BF16 = 0, 1
BUCKET_MOD, BUCKET_HASH = 0, 1
NORM_NONE, NORM_MEAN = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2
USER_RAW, USER_PROJECTED = 0, 1
NOALLOC_MAX_CANDIDATES, NOALLOC_ROW_BYTES = 1024, 4096
BLK_ATT, BLK_CROSS, BLK_BEA, BLK_LSH_DIN, BLK_SIMTIER = 1, 2, 4, 8, 16


class AifError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {_strerror(code)} ({code}) {detail}".strip())


class aif_config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("dtype", C.c_int32), ("M", C.c_int64), ("d", C.c_int32), ("dU", C.c_int32),
        ("L_max", C.c_int32), ("F", C.c_int32), ("B", C.c_int32), ("dc", C.c_int32), ("n_hidden", C.c_int32),
        ("hidden", C.c_int32 * 4), ("bucket_mode", C.c_int32), ("blocks", C.c_int32), ("n_bridge", C.c_int32),
        ("lsh_bits", C.c_int32), ("n_tiers", C.c_int32), ("lsh_din_norm", C.c_int32), ("simtier_norm", C.c_int32),
        ("emit_sigmoid", C.c_int32), ("max_user_states", C.c_int32), ("mini_batch", C.c_int32), ("path", C.c_int32),
        ("n_categories", C.c_int32), ("versioned_table", C.c_int32), ("max_batch_candidates", C.c_int64),
    ]


class aif_weights(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("W", C.c_void_p * 4), ("b", C.c_void_p * 4), ("w_out", C.c_void_p),
        ("b_out", C.c_void_p), ("W_profile", C.c_void_p), ("W_seq", C.c_void_p), ("W_a", C.c_void_p),
        ("b_a", C.c_void_p), ("W_b", C.c_void_p), ("b_b", C.c_void_p), ("bridges", C.c_void_p), ("W_f", C.c_void_p),
    ]


class aif_item_weights(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("dI", C.c_int32), ("hI", C.c_int32), ("d_mm", C.c_int32), ("W_i0", C.c_void_p),
        ("b_i0", C.c_void_p), ("W_i1", C.c_void_p), ("b_i1", C.c_void_p), ("bridges", C.c_void_p), ("W_hash", C.c_void_p),
    ]


class aif_user_inputs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("mode", C.c_int32), ("profile", C.c_void_p), ("seq", C.c_void_p),
        ("cross_raw", C.c_void_p), ("bea_V", C.c_void_p), ("seq_sig", C.c_void_p), ("bea_U", C.c_void_p), ("seq_cat", C.c_void_p),
        ("bea_m", C.c_int32),
    ]


class aif_stats(C.Structure):
    _fields_ = [
        ("score_calls", C.c_uint64), ("candidates_scored", C.c_uint64), ("precompute_calls", C.c_uint64),
        ("refresh_calls", C.c_uint64), ("rows_refreshed", C.c_uint64), ("bad_id_events", C.c_uint64),
        ("timeout_events", C.c_uint64), ("user_states_in_use", C.c_int32), ("user_states_high_water", C.c_int32),
        ("model_version", C.c_uint64), ("table_version", C.c_uint64), ("device_bytes", C.c_int64),
        ("tensor_path", C.c_int32),
    ]


# every symbol include/aif.h declares
EXPORTS = [
    "aif_input_width", "aif_mix64", "aif_category", "aif_create", "aif_destroy", "aif_load_weights", "aif_item_nearline_refresh",
    "aif_load_item_weights", "aif_item_nearline_compute",
    "aif_user_precompute", "aif_user_release", "aif_user_request_key", "aif_user_state_export", "aif_user_state_export_bea", "aif_score",
    "aif_score_batch", "aif_score_host", "aif_score_batch_host", "aif_score_noalloc", "aif_gather_rows", "aif_gather_sidecars", "aif_poll_status", "aif_get_stats",
    "aif_set_kernel_timing", "aif_get_kernel_timing", "aif_kernel_launches", "aif_selftest_bounded_wait", "aif_strerror", "aif_last_error",
]

_lib = None


def load_library(path: Optional[str] = None):
    """Loads libaif.so; raises if it is missing (build it with paper_2511_12934_b200/build.py)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: the CUDA library is not built and there is no fallback")
    lib = C.CDLL(p)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    lib.aif_input_width.argtypes = [C.POINTER(aif_config)]
    lib.aif_mix64.argtypes, lib.aif_mix64.restype = [u64, u64], u64
    lib.aif_category.argtypes, lib.aif_category.restype = [i64, i32, i32], i64
    lib.aif_create.argtypes = [C.POINTER(aif_config), C.POINTER(vp)]
    lib.aif_destroy.argtypes = [vp]
    lib.aif_load_weights.argtypes = [vp, C.POINTER(aif_weights), vp]
    lib.aif_item_nearline_refresh.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.aif_load_item_weights.argtypes = [vp, C.POINTER(aif_item_weights), vp]
    lib.aif_item_nearline_compute.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.aif_user_precompute.argtypes = [vp, u64, C.POINTER(aif_user_inputs), i32, C.POINTER(vp), vp]
    lib.aif_user_release.argtypes = [vp, vp]
    lib.aif_user_request_key.argtypes, lib.aif_user_request_key.restype = [vp], u64
    lib.aif_user_state_export.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.aif_user_state_export_bea.argtypes = [vp, vp, vp, vp]
    lib.aif_score.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.aif_score_batch.argtypes = [vp, i32, C.POINTER(vp), vp, C.POINTER(i64), vp, vp]
    lib.aif_score_host.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.aif_score_batch_host.argtypes = [vp, i32, C.POINTER(vp), vp, C.POINTER(i64), vp, vp]
    lib.aif_score_noalloc.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.aif_gather_rows.argtypes = [vp, vp, i64, vp, vp]
    lib.aif_gather_sidecars.argtypes = [vp, vp, i64, vp, vp, vp]
    lib.aif_poll_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.aif_get_stats.argtypes = [vp, C.POINTER(aif_stats)]
    lib.aif_set_kernel_timing.argtypes = [vp, C.c_int]
    lib.aif_get_kernel_timing.argtypes = [vp, C.POINTER(i32), C.POINTER(C.c_char_p), C.POINTER(C.c_float)]
    lib.aif_kernel_launches.argtypes, lib.aif_kernel_launches.restype = [], u64
    lib.aif_selftest_bounded_wait.argtypes = [vp, i64, vp]
    lib.aif_strerror.argtypes, lib.aif_strerror.restype = [C.c_int], C.c_char_p
    lib.aif_last_error.argtypes, lib.aif_last_error.restype = [], C.c_char_p
    if path is None:
        _lib = lib
    return lib


def _strerror(code: int) -> str:
    try:
        return load_library().aif_strerror(code).decode()
    except Exception:
        return "error"


def _check(rc: int, where: str):
    if rc != OK:
        raise AifError(rc, where, load_library().aif_last_error().decode())


def mix64(id_: int, field: int) -> int:
    return int(load_library().aif_mix64(id_, field))


def kernel_launches() -> int:
    return int(load_library().aif_kernel_launches())


def to_device(a: np.ndarray, dtype: int, device="cuda") -> torch.Tensor:
    """Storage array (float32, or uint16 bf16 bit patterns) -> device tensor of the matching torch type."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16 and dtype == BF16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream(s) -> C.c_void_p:
    if s is None:
        s = torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_config(*, dtype, M, d, L_max, hidden: Sequence[int], F=0, B=1, dc=0, dU=0, bucket_mode=BUCKET_HASH,
                blocks=BLK_ATT | BLK_CROSS, n_bridge=8, lsh_bits=0, n_tiers=8, lsh_din_norm=NORM_MEAN,
                simtier_norm=NORM_MEAN, emit_sigmoid=0, max_user_states=4, mini_batch=0, path=PATH_AUTO,
                max_batch_candidates=16384, n_categories=0, versioned_table=0) -> aif_config:
    h = list(hidden) + [0] * (4 - len(hidden))
    return aif_config(C.sizeof(aif_config), dtype, M, d, dU or d, L_max, F, B, dc, len(hidden), (C.c_int32 * 4)(*h),
                      bucket_mode, blocks, n_bridge, lsh_bits or d, n_tiers, lsh_din_norm, simtier_norm,
                      emit_sigmoid, max_user_states, mini_batch, path, n_categories, versioned_table, max_batch_candidates)


class UserState:
    """Handle of one slot of the user-state arena."""

    def __init__(self, ctx: "Aif", handle: int, keep):
        self.ctx, self.handle, self._keep = ctx, handle, keep

    @property
    def request_key(self) -> int:
        return int(self.ctx.lib.aif_user_request_key(self.handle))

    def release(self):
        if self.handle:
            _check(self.ctx.lib.aif_user_release(self.ctx.h, self.handle), "aif_user_release")
            self.handle = None


class Aif:
    """One libaif context on the current CUDA device."""

    def __init__(self, cfg: aif_config):
        if not torch.cuda.is_available():
            raise RuntimeError("libaif needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.cfg = cfg
        h = C.c_void_p()
        _check(self.lib.aif_create(C.byref(cfg), C.byref(h)), "aif_create")
        self.h = h
        self.torch_dtype = torch.float32 if cfg.dtype == F32 else torch.bfloat16
        self._weights_keep = None

    def close(self):
        if self.h:
            self.lib.aif_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def input_width(self) -> int:
        return int(self.lib.aif_input_width(C.byref(self.cfg)))

    # -- weights ---------------------------------------------------------------------------------
    def load_weights(self, mlp: dict, user: Optional[dict] = None, stream=None):
        """mlp: {"W": [..], "b": [..], "w_out", "b_out"}; user: {"W_profile", "W_seq", "W_a", "b_a", "W_b", "b_b"};
        values are device tensors (weights in storage type, biases fp32)."""
        w = aif_weights()
        w.struct_size = C.sizeof(aif_weights)
        for k in range(self.cfg.n_hidden):
            w.W[k] = mlp["W"][k].data_ptr()
            w.b[k] = mlp["b"][k].data_ptr()
        w.w_out, w.b_out = mlp["w_out"].data_ptr(), mlp["b_out"].data_ptr()
        if user is not None:
            for name in ("W_profile", "W_seq", "W_a", "b_a", "W_b", "b_b", "bridges", "W_f"):
                if user.get(name) is not None:
                    setattr(w, name, user[name].data_ptr())
        _check(self.lib.aif_load_weights(self.h, C.byref(w), _stream(stream)), "aif_load_weights")
        self._weights_keep = (mlp, user)

    def load_weights_host(self, weights: dict):
        """Convenience: weights as produced by synth.make_weights (host storage arrays)."""
        dt = self.cfg.dtype
        mlp = weights["mlp"]
        dm = {"W": [to_device(a, dt) for a in mlp["W"]], "b": [torch.from_numpy(a).cuda() for a in mlp["b"]],
              "w_out": to_device(mlp["w_out"], dt), "b_out": torch.from_numpy(mlp["b_out"]).cuda()}
        du = None
        if weights.get("user") is not None:
            u = weights["user"]
            du = {k: (torch.from_numpy(v).cuda() if k.startswith("b_") else to_device(v, dt)) for k, v in u.items()}
        self.load_weights(dm, du)
        torch.cuda.current_stream().synchronize()

    # -- item side -------------------------------------------------------------------------------
    def item_nearline_refresh(self, ids: Optional[torch.Tensor], rows: torch.Tensor, bea_w=None, lsh_sig=None,
                              stream=None):
        n = rows.shape[0]
        _check(self.lib.aif_item_nearline_refresh(self.h, _ptr(ids), n, _ptr(rows), _ptr(bea_w), _ptr(lsh_sig),
                                                  _stream(stream)), "aif_item_nearline_refresh")

    def load_item_weights(self, w: dict, stream=None):
        """w: device tensors "W_i0" [hI x dI], "b_i0", "W_i1" [d x hI], "b_i1" and, for their blocks, "bridges"
        [n_bridge x d], "W_hash" [lsh_bits x d_mm] (weights in storage type, biases fp32)."""
        iw = aif_item_weights()
        iw.struct_size = C.sizeof(aif_item_weights)
        iw.hI, iw.dI = w["W_i0"].shape
        iw.d_mm = w["W_hash"].shape[1] if w.get("W_hash") is not None else 0
        for name in ("W_i0", "b_i0", "W_i1", "b_i1", "bridges", "W_hash"):
            if w.get(name) is not None:
                setattr(iw, name, w[name].data_ptr())
        _check(self.lib.aif_load_item_weights(self.h, C.byref(iw), _stream(stream)), "aif_load_item_weights")
        self._item_weights_keep = w

    def item_nearline_compute(self, ids: Optional[torch.Tensor], I_raw: torch.Tensor, I_id=None, M_mm=None, stream=None):
        _check(self.lib.aif_item_nearline_compute(self.h, _ptr(ids), I_raw.shape[0], _ptr(I_raw), _ptr(I_id), _ptr(M_mm),
                                                  _stream(stream)), "aif_item_nearline_compute")

    def gather_rows(self, ids: torch.Tensor, out: torch.Tensor, stream=None):
        _check(self.lib.aif_gather_rows(self.h, _ptr(ids), ids.numel(), _ptr(out), _stream(stream)), "aif_gather_rows")

    def user_state_export_bea(self, state: "UserState", stream=None) -> torch.Tensor:
        V = torch.empty(self.cfg.n_bridge, self.cfg.d, dtype=self.torch_dtype, device="cuda")
        _check(self.lib.aif_user_state_export_bea(self.h, state.handle, _ptr(V), _stream(stream)), "aif_user_state_export_bea")
        return V

    def gather_sidecars(self, ids: torch.Tensor, bea_w_out=None, sig_out=None, stream=None):
        _check(self.lib.aif_gather_sidecars(self.h, _ptr(ids), ids.numel(), _ptr(bea_w_out), _ptr(sig_out), _stream(stream)),
               "aif_gather_sidecars")

    # -- user side -------------------------------------------------------------------------------
    def user_precompute(self, request_key: int, *, mode: int, profile: torch.Tensor, seq: torch.Tensor,
                        cross_raw=None, bea_V=None, seq_sig=None, bea_U=None, seq_cat=None, stream=None) -> UserState:
        inp = aif_user_inputs(C.sizeof(aif_user_inputs), mode, profile.data_ptr(), seq.data_ptr(),
                              None if cross_raw is None else cross_raw.data_ptr(),
                              None if bea_V is None else bea_V.data_ptr(),
                              None if seq_sig is None else seq_sig.data_ptr(),
                              None if bea_U is None else bea_U.data_ptr(), None if seq_cat is None else seq_cat.data_ptr(),
                              0 if bea_U is None else bea_U.shape[0])
        out = C.c_void_p()
        _check(self.lib.aif_user_precompute(self.h, request_key, C.byref(inp), seq.shape[0], C.byref(out),
                                            _stream(stream)), "aif_user_precompute")
        return UserState(self, out.value, (profile, seq, cross_raw, bea_V, seq_sig, bea_U, seq_cat))

    def user_state_export(self, state: UserState, L: int, stream=None):
        u = torch.empty(self.cfg.d, dtype=torch.float32, device="cuda")
        S = torch.empty(L, self.cfg.d, dtype=self.torch_dtype, device="cuda")
        pu = torch.empty(self.cfg.hidden[0], dtype=torch.float32, device="cuda")
        _check(self.lib.aif_user_state_export(self.h, state.handle, _ptr(u), _ptr(S), _ptr(pu), _stream(stream)),
               "aif_user_state_export")
        return u, S, pu

    # -- real time -------------------------------------------------------------------------------
    def score(self, state: UserState, cand_ids: torch.Tensor, logits: torch.Tensor, stream=None):
        _check(self.lib.aif_score(self.h, state.handle, _ptr(cand_ids), cand_ids.numel(), _ptr(logits),
                                  _stream(stream)), "aif_score")

    def score_noalloc(self, state: UserState, cand_ids: torch.Tensor, logits: torch.Tensor, stream=None):
        """aif_score_noalloc: same arguments as score; activations live in the library's fixed device array."""
        _check(self.lib.aif_score_noalloc(self.h, state.handle, _ptr(cand_ids), cand_ids.numel(), _ptr(logits),
                                          _stream(stream)), "aif_score_noalloc")

    def score_batch(self, states: Sequence[UserState], cand_ids: torch.Tensor, offsets: Sequence[int],
                    logits: torch.Tensor, stream=None):
        n = len(states)
        hs = (C.c_void_p * n)(*[s.handle for s in states])
        off = (C.c_int64 * (n + 1))(*[int(o) for o in offsets])
        _check(self.lib.aif_score_batch(self.h, n, hs, _ptr(cand_ids), off, _ptr(logits), _stream(stream)),
               "aif_score_batch")

    def score_host(self, state: UserState, host_ids: torch.Tensor, host_logits: torch.Tensor, stream=None):
        """host_ids int32 / host_logits float32: CPU tensors (pinned for best speed)."""
        assert not host_ids.is_cuda and not host_logits.is_cuda
        _check(self.lib.aif_score_host(self.h, state.handle, C.c_void_p(host_ids.data_ptr()), host_ids.numel(),
                                       C.c_void_p(host_logits.data_ptr()), _stream(stream)), "aif_score_host")

    def score_batch_host(self, states: Sequence[UserState], host_ids: torch.Tensor, offsets: Sequence[int],
                         host_logits: torch.Tensor, stream=None):
        """aif_score_batch with CPU tensors (int32 ids of all requests concatenated, float32 logits)."""
        assert not host_ids.is_cuda and not host_logits.is_cuda
        n = len(states)
        hs = (C.c_void_p * n)(*[s.handle for s in states])
        off = (C.c_int64 * (n + 1))(*[int(o) for o in offsets])
        _check(self.lib.aif_score_batch_host(self.h, n, hs, C.c_void_p(host_ids.data_ptr()), off,
                                             C.c_void_p(host_logits.data_ptr()), _stream(stream)), "aif_score_batch_host")

    # -- status ----------------------------------------------------------------------------------
    def poll_status(self) -> int:
        bits = C.c_uint32()
        _check(self.lib.aif_poll_status(self.h, C.byref(bits)), "aif_poll_status")
        return int(bits.value)

    def selftest_bounded_wait(self, limit_cycles: int, stream=None):
        """Launches the kernel whose only wait runs out after limit_cycles; poll_status then shows STATUS_TIMEOUT."""
        _check(self.lib.aif_selftest_bounded_wait(self.h, int(limit_cycles), _stream(stream)), "aif_selftest_bounded_wait")

    def set_kernel_timing(self, on: bool):
        _check(self.lib.aif_set_kernel_timing(self.h, 1 if on else 0), "aif_set_kernel_timing")

    def get_kernel_timing(self) -> dict:
        """{kernel name: milliseconds} of the last scoring call (timing must be on)."""
        n = C.c_int32()
        names = (C.c_char_p * 8)()
        ms = (C.c_float * 8)()
        _check(self.lib.aif_get_kernel_timing(self.h, C.byref(n), names, ms), "aif_get_kernel_timing")
        return {names[i].decode(): float(ms[i]) for i in range(n.value)}

    def get_stats(self) -> aif_stats:
        s = aif_stats()
        _check(self.lib.aif_get_stats(self.h, C.byref(s)), "aif_get_stats")
        return s
