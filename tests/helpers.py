"""Glue shared by the tests: maps a synthetic workload onto the oracle's configuration."""
import numpy as np

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import synth


def oracle_config(wl: synth.Workload, M=None) -> orc.OracleConfig:
    return orc.OracleConfig(
        dtype=orc.F32 if wl.dtype == "f32" else orc.BF16, M=M or wl.M, d=wl.d, F=wl.F, B=wl.B, dc=wl.dc,
        hidden=tuple(wl.hidden), bucket_mode=wl.bucket_mode, blocks=wl.blocks, n_bridge=wl.n_bridge,
        lsh_bits=wl.lsh_bits, n_tiers=wl.n_tiers, lsh_din_norm=wl.lsh_din_norm, simtier_norm=wl.simtier_norm,
        emit_sigmoid=wl.emit_sigmoid, n_categories=wl.n_categories)


def make_oracle(wl: synth.Workload, weights: dict, M=None) -> orc.Oracle:
    return orc.Oracle(oracle_config(wl, M), weights["mlp"], weights["user"])


def projected_request(wl: synth.Workload, rq: dict) -> dict:
    """Request dict for Oracle.score when the caller supplies u and S directly."""
    out = {"u": synth.as_f32(rq["u"], wl.dtype).astype(np.float64),
           "S": synth.as_f32(rq["S"], wl.dtype).astype(np.float64)}
    for k in ("T", "V", "sig_seq", "seq_cat"):
        if k in rq:
            out[k] = rq[k]
    return out


def raw_request(oracle: orc.Oracle, rq: dict) -> dict:
    """Request dict for Oracle.score with u and S computed by the oracle's user-side network (eqs. 1-3)."""
    u, S = oracle.user_state(rq["profile"], rq["seq"])
    out = {"u": u, "S": S}
    for k in ("T", "V", "sig_seq", "seq_cat"):
        if k in rq:
            out[k] = rq[k]
    return out


ALL_BLOCKS = synth.BLK_ATT | synth.BLK_CROSS | synth.BLK_BEA | synth.BLK_LSH_DIN | synth.BLK_SIMTIER

# Scaled-down copies of the five shapes: every dimension that changes code paths is kept (dtype, bucket mode,
# number of layers, d, dc), sizes are cut so that the oracle finishes in seconds, candidate counts span
# several 128-row tiles and leave a ragged tail.
MINI = {
    "c1": synth.C1.with_(name="mini_c1", N=301, M=5000),
    "c2": synth.C2.with_(name="mini_c2", N=1100, M=20000, mini_batch=500),
    "c3": synth.C3.with_(name="mini_c3", R=3, N=333, M=30000, L=300),
    "c4": synth.C4.with_(name="mini_c4", R=2, N=200, M=20000, L=1100),
    "c5": synth.C5.with_(name="mini_c5", R=3, N=260, M=10000, L=130, F=64, B=4096),
}
