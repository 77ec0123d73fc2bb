"""Request-level glue around the binding: builds a context for a synthetic workload, fills the item table through
aif_item_nearline_refresh, and runs the two calls of a request (user precompute on a side stream, then scoring).
No arithmetic of the method lives here."""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import synth


def config_for(wl: synth.Workload, *, rows: Optional[int] = None, L_max: Optional[int] = None,
               max_user_states: Optional[int] = None, path: int = B.PATH_AUTO,
               max_batch_candidates: Optional[int] = None, versioned_table: int = 0) -> B.aif_config:
    dt = B.F32 if wl.dtype == "f32" else B.BF16
    return B.make_config(
        dtype=dt, M=rows or wl.M, d=wl.d, L_max=L_max or wl.L, hidden=wl.hidden, F=wl.F, B=wl.B, dc=wl.dc,
        dU=wl.raw_dU, bucket_mode=wl.bucket_mode, blocks=wl.blocks, n_bridge=wl.n_bridge, lsh_bits=wl.lsh_bits,
        n_tiers=wl.n_tiers, lsh_din_norm=wl.lsh_din_norm, simtier_norm=wl.simtier_norm,
        emit_sigmoid=wl.emit_sigmoid, max_user_states=max_user_states or max(2, wl.R), mini_batch=wl.mini_batch,
        path=path, max_batch_candidates=max_batch_candidates or max(1, wl.R * wl.N), n_categories=wl.n_categories,
        versioned_table=versioned_table)


class Server:
    """A context loaded with a workload's weights and item table."""

    def __init__(self, wl: synth.Workload, weights: dict, table: dict, **cfg_kw):
        self.wl = wl
        self.cfg = config_for(wl, rows=table["E"].shape[0], **cfg_kw)
        self.ctx = B.Aif(self.cfg)
        self.dt = self.cfg.dtype
        self.ctx.load_weights_host(weights)
        self.side = torch.cuda.Stream()
        self.refresh_full(table)

    def refresh_full(self, table: dict):
        E = B.to_device(table["E"], self.dt)
        bw = B.to_device(table["bea_w"], self.dt) if "bea_w" in table else None
        sg = torch.from_numpy(np.ascontiguousarray(table["sig"])).cuda() if "sig" in table else None
        self.ctx.item_nearline_refresh(None, E, bw, sg)
        torch.cuda.synchronize()

    def refresh_rows(self, ids: np.ndarray, rows: np.ndarray, bea_w=None, sig=None):
        ids_t = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda()
        self.ctx.item_nearline_refresh(
            ids_t, B.to_device(rows, self.dt), None if bea_w is None else B.to_device(bea_w, self.dt),
            None if sig is None else torch.from_numpy(np.ascontiguousarray(sig)).cuda())
        torch.cuda.synchronize()

    def upload_request(self, rq: dict, mode: int) -> dict:
        """Host request dict (synth.make_request) -> device tensors for aif_user_precompute."""
        dev = {"mode": mode}
        if mode == B.USER_RAW:
            dev["profile"], dev["seq"] = B.to_device(rq["profile"], self.dt), B.to_device(rq["seq"], self.dt)
        else:
            dev["profile"], dev["seq"] = B.to_device(rq["u"], self.dt), B.to_device(rq["S"], self.dt)
        dev["cross_raw"] = B.to_device(rq["T"], self.dt) if "T" in rq else None
        dev["bea_V"] = B.to_device(rq["V"], self.dt) if "V" in rq else None
        dev["bea_U"] = B.to_device(rq["bea_U"], self.dt) if "bea_U" in rq else None   # Algorithm 1's U: V is computed
        dev["seq_sig"] = torch.from_numpy(np.ascontiguousarray(rq["sig_seq"])).cuda() if "sig_seq" in rq else None
        dev["seq_cat"] = torch.from_numpy(np.ascontiguousarray(rq["seq_cat"], dtype=np.int32)).cuda() if "seq_cat" in rq else None
        return dev

    def precompute(self, key: int, dev: dict, stream=None) -> B.UserState:
        """aif_user_precompute on the side stream (or `stream`)."""
        return self.ctx.user_precompute(key, mode=dev["mode"], profile=dev["profile"], seq=dev["seq"],
                                        cross_raw=dev["cross_raw"], bea_V=dev["bea_V"], seq_sig=dev["seq_sig"],
                                        bea_U=dev.get("bea_U"), seq_cat=dev.get("seq_cat"), stream=stream or self.side)

    def score_ids(self, state: B.UserState, ids: np.ndarray) -> np.ndarray:
        ids_t = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).cuda()
        out = torch.empty(ids_t.numel(), dtype=torch.float32, device="cuda")
        self.ctx.score(state, ids_t, out)
        torch.cuda.synchronize()
        return out.cpu().numpy()

    def score_many(self, states: Sequence[B.UserState], id_lists: Sequence[np.ndarray]):
        offs = np.zeros(len(id_lists) + 1, dtype=np.int64)
        offs[1:] = np.cumsum([len(x) for x in id_lists])
        ids_t = torch.from_numpy(np.ascontiguousarray(np.concatenate(id_lists), dtype=np.int32)).cuda()
        out = torch.empty(ids_t.numel(), dtype=torch.float32, device="cuda")
        self.ctx.score_batch(states, ids_t, offs, out)
        torch.cuda.synchronize()
        o = out.cpu().numpy()
        return [o[offs[i]:offs[i + 1]] for i in range(len(id_lists))]

    def close(self):
        self.ctx.close()
