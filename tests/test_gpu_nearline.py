"""Item side of the nearline pipeline as a compute call (aif_item_nearline_compute) against the CPU oracle: item vectors
(Section 3.2 eq. 4), BEA weight rows (Algorithm 1 step 3) and LSH signatures (Section 4.2 eq. 5), full and incremental."""
import numpy as np
import pytest
import torch

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import binding as B
from paper_2511_12934_b200 import build as libbuild
from paper_2511_12934_b200 import serving, synth
from tests import helpers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    B.load_library()


def _read_back(srv, wl, ids):
    ids_t = torch.from_numpy(ids.astype(np.int32)).cuda()
    tdt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    rows = torch.empty(len(ids), wl.d, dtype=tdt, device="cuda")
    bea = torch.empty(len(ids), wl.n_bridge, dtype=tdt, device="cuda")
    sig = torch.empty(len(ids), wl.lsh_bits // 8, dtype=torch.uint8, device="cuda")
    srv.ctx.gather_rows(ids_t, rows)
    srv.ctx.gather_sidecars(ids_t, bea, sig)
    torch.cuda.synchronize()
    return rows.float().cpu().numpy().astype(np.float64), bea.float().cpu().numpy().astype(np.float64), sig.cpu().numpy()


# widths: (dI, hI, d_mm).  bf16 with multiples of 64 runs on the tensor cores: hidden widths up to 256 at d = 128 in the
# one-kernel tower (ragged last tile, an odd number of tiles, more tile pairs than one CTA round at M = 4000 is not needed:
# pairs are walked persistently), wider ones and d = 256 as two launches of the layer kernel; the other shapes run the
# CUDA-core kernels.
@pytest.mark.parametrize("name,dims,n", [("c1", (40, 24, 20), 777), ("c2", (512, 256, 128), 1111), ("c2", (192, 512, 64), 300),
                                         ("c2", (100, 60, 36), 333), ("c5", (256, 128, 256), 515), ("c2", (128, 192, 128), 3000),
                                         ("c2", (64, 64, 64), 130)])
@pytest.mark.parametrize("incremental", [False, True])
def test_nearline_compute_matches_the_oracle(name, dims, n, incremental):
    dI, hI, d_mm = dims
    wl = helpers.MINI[name].with_(name=f"nearline_{name}", blocks=helpers.ALL_BLOCKS, M=4000, L=20, N=50)
    weights = synth.make_weights(wl)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table)
    dt = orc.F32 if wl.dtype == "f32" else orc.BF16
    bdt = B.F32 if wl.dtype == "f32" else B.BF16
    it = synth.make_item_side(wl, n, dI, hI, d_mm)
    dev = {k: (torch.from_numpy(v).cuda() if v.dtype == np.float32 else B.to_device(v, bdt)) for k, v in it.items()}
    srv.ctx.load_item_weights(dev)
    if incremental:
        g = np.random.default_rng(5)
        ids = g.choice(wl.M, n, replace=False).astype(np.int32)
        ids[7], ids[100] = -1, wl.M + 3
        srv.ctx.item_nearline_compute(torch.from_numpy(ids).cuda(), dev["I_raw"], dev["I_id"], dev["M_mm"])
        assert srv.ctx.poll_status() == B.STATUS_BAD_ID
        good = (ids >= 0) & (ids < wl.M)
    else:
        ids = np.arange(n, dtype=np.int32)
        srv.ctx.item_nearline_compute(None, dev["I_raw"], dev["I_id"], dev["M_mm"])
        assert srv.ctx.poll_status() == 0
        good = np.ones(n, dtype=bool)
    want = orc.item_nearline(dt, I_raw=it["I_raw"], W0=it["W_i0"], b0=it["b_i0"], W1=it["W_i1"], b1=it["b_i1"], I_id=it["I_id"],
                             bridges=it["bridges"], M_mm=it["M_mm"], W_hash=it["W_hash"])
    rows, bea, sig = _read_back(srv, wl, np.where(good, ids, 0))
    rows, bea, sig = rows[good], bea[good], sig[good]
    # item vectors: fp32 arithmetic, or bf16 hidden activations and bf16 storage (relative 2^-9 each)
    rtol, atol = (1e-5, 1e-6) if wl.dtype == "f32" else (2.0 ** -7, 5e-4)
    assert np.allclose(rows, want["I_hat"][good], rtol=rtol, atol=atol), np.abs(rows - want["I_hat"][good]).max()
    # bridge weights: a softmax row, stored in the table's type
    assert np.allclose(bea, want["w_hat"][good], rtol=rtol, atol=1e-6 if wl.dtype == "f32" else 2.0 ** -9)
    # signatures: bit for bit, except bits whose projection is within rounding of zero (fp32 sums of d_mm products of
    # O(1) values in another order); those must be few
    proj = orc.lsh_projections(dt, it["M_mm"], it["W_hash"])[good]
    got_bits = np.unpackbits(sig, axis=1, bitorder="big")
    want_bits = np.unpackbits(want["sig"][good], axis=1, bitorder="big")
    differ = got_bits != want_bits
    assert np.all(np.abs(proj[differ]) < 1e-4 * np.sqrt(d_mm)), np.abs(proj[differ]).max()
    assert differ.mean() < 1e-4
    # rows that were not addressed keep their old contents
    if incremental:
        others = np.setdiff1d(np.arange(wl.M), ids[good])[:200].astype(np.int32)
        old_rows, _, old_sig = _read_back(srv, wl, others)
        assert np.array_equal(old_rows, synth.as_f32(table["E"][others], wl.dtype).astype(np.float64))
        assert np.array_equal(old_sig, table["sig"][others])
    srv.close()


def test_one_kernel_tower_with_several_tile_pairs_per_cta():
    """More rows than 148 CTAs take in one round of tile pairs (each CTA walks over three pairs, the last one ragged):
    the reuse of tensor memory, of the barriers' phases and of the operand rings from pair to pair."""
    n = 148 * 256 * 2 + 9 * 256 + 77
    wl = helpers.MINI["c2"].with_(name="nearline_pairs", M=n, L=20, N=50)
    srv = serving.Server(wl, synth.make_weights(wl), {"E": np.zeros((n, wl.d), dtype=np.uint16)})
    it = synth.make_item_side(wl, n, 128, 128, 64)
    dev = {k: (torch.from_numpy(v).cuda() if v.dtype == np.float32 else B.to_device(v, B.BF16)) for k, v in it.items()}
    srv.ctx.load_item_weights(dev)
    srv.ctx.item_nearline_compute(None, dev["I_raw"])
    assert srv.ctx.poll_status() == 0
    want = orc.item_nearline(orc.BF16, I_raw=it["I_raw"], W0=it["W_i0"], b0=it["b_i0"], W1=it["W_i1"], b1=it["b_i1"])["I_hat"]
    ids_t = torch.arange(n, dtype=torch.int32, device="cuda")
    rows = torch.empty(n, wl.d, dtype=torch.bfloat16, device="cuda")
    srv.ctx.gather_rows(ids_t, rows)
    torch.cuda.synchronize()
    got = rows.float().cpu().numpy().astype(np.float64)
    assert np.allclose(got, want, rtol=2.0 ** -7, atol=5e-4), np.abs(got - want).max()
    srv.close()


def test_scoring_on_a_table_built_by_the_nearline_call():
    """End to end: the table rows come from aif_item_nearline_compute, the scores from aif_score; the oracle does both
    from the same raw inputs.  The item vectors differ from the oracle's by bf16 rounding, so the budget is the bf16
    logit tolerance plus that rounding carried through the first layer."""
    wl = helpers.MINI["c2"].with_(name="nearline_e2e", blocks=helpers.ALL_BLOCKS, M=3000, N=400, L=60,
                                  lsh_din_norm=synth.NORM_MEAN, simtier_norm=synth.NORM_MEAN)
    weights = synth.make_weights(wl)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table)
    it = synth.make_item_side(wl, wl.M)
    dev = {k: (torch.from_numpy(v).cuda() if v.dtype == np.float32 else B.to_device(v, B.BF16)) for k, v in it.items()}
    srv.ctx.load_item_weights(dev)
    srv.ctx.item_nearline_compute(None, dev["I_raw"], dev["I_id"], dev["M_mm"])
    want_tab = orc.item_nearline(orc.BF16, I_raw=it["I_raw"], W0=it["W_i0"], b0=it["b_i0"], W1=it["W_i1"], b1=it["b_i1"],
                                 I_id=it["I_id"], bridges=it["bridges"], M_mm=it["M_mm"], W_hash=it["W_hash"])
    host = {"E": synth.to_bf16_bits(want_tab["I_hat"].astype(np.float32)), "bea_w": synth.to_bf16_bits(want_tab["w_hat"].astype(np.float32)),
            "sig": want_tab["sig"]}
    oracle = helpers.make_oracle(wl, weights, M=wl.M)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want = oracle.score(host, helpers.projected_request(wl, rq), ids)
    got = srv.score_ids(st, ids)
    assert np.abs(got - want).max() <= 4e-3
    srv.close()


@pytest.mark.parametrize("dims", [(512, 256, 64), (192, 512, 64)])
def test_item_vectors_from_the_nearline_call_raise_the_tables_norm_bound(dims):
    """The attention kernel drops its running maximum only while (largest item norm) x (largest sequence-row norm) keeps
    the scores within 2^+-50; the nearline call has to raise the table's bound from the rows it computes (inside the
    one-kernel tower for the first shape, by a pass over its output for the second).  The table starts with small
    vectors; the call then writes vectors with every component near 40, and the sequence is scaled so that scores reach
    several hundred: scored with a stale bound the exponentials overflow.  The oracle scores on the rows read back from
    the device (the item side's own parity is checked elsewhere)."""
    wl = helpers.MINI["c2"].with_(name=f"nearline_norm_{dims[1]}", M=2000, N=500, L=300, mini_batch=0, hidden=(256, 256))
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table)
    it = synth.make_item_side(wl, wl.M, dI=dims[0], hI=dims[1], d_mm=dims[2])
    it["b_i1"] = (it["b_i1"] + 40.0).astype(np.float32)
    dev = {k: (torch.from_numpy(v).cuda() if v.dtype == np.float32 else B.to_device(v, B.BF16)) for k, v in it.items()}
    srv.ctx.load_item_weights(dev)
    srv.ctx.item_nearline_compute(None, dev["I_raw"], dev["I_id"], dev["M_mm"])
    ids_all = torch.arange(wl.M, dtype=torch.int32, device="cuda")
    rows = torch.empty(wl.M, wl.d, dtype=torch.bfloat16, device="cuda")
    srv.ctx.gather_rows(ids_all, rows)
    torch.cuda.synchronize()
    host = {"E": rows.view(torch.int16).cpu().numpy().view(np.uint16)}
    assert np.abs(synth.bf16_bits_to_f32(host["E"])).mean() > 30.0
    rq = synth.make_request(wl, 0)
    rq["S"] = synth.to_bf16_bits(synth.bf16_bits_to_f32(rq["S"]) * 16.0)
    oracle = helpers.make_oracle(wl, weights, M=wl.M)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want, x = oracle.score(host, helpers.projected_request(wl, rq), ids, return_inputs=True)
    got = srv.score_ids(st, ids)
    assert np.isfinite(got).all()
    # bf16 intermediates of magnitude A carry about 2^-9 A of rounding error: the budget follows the MLP's inputs (about 40)
    assert np.abs(got - want).max() <= 2e-3 * max(1.0, float(np.abs(x).max()))
    assert srv.ctx.get_stats().tensor_path == 1 and srv.ctx.poll_status() == 0
    srv.close()


def test_nearline_call_errors():
    wl = helpers.MINI["c1"].with_(name="nearline_err", M=500)
    srv = serving.Server(wl, synth.make_weights(wl), synth.make_item_table(wl))
    x = torch.zeros(10, 40, device="cuda")
    with pytest.raises(B.AifError) as e:
        srv.ctx.item_nearline_compute(None, x)
    assert e.value.code == B.ERR_NOT_READY
    it = synth.make_item_side(wl, 10, 40, 24, 20)
    dev = {k: torch.from_numpy(v).cuda() for k, v in it.items()}
    srv.ctx.load_item_weights(dev)
    srv.ctx.item_nearline_compute(None, dev["I_raw"])          # blocks off: no sidecar inputs needed
    with pytest.raises(B.AifError) as e:
        srv.ctx.item_nearline_compute(None, torch.zeros(501, 40, device="cuda"))
    assert e.value.code == B.ERR_SHAPE
    bad = dict(dev, W_i0=torch.zeros(24, 44, device="cuda"))   # other widths than the first call's
    with pytest.raises(B.AifError) as e:
        srv.ctx.load_item_weights(bad)
    assert e.value.code == B.ERR_SHAPE
    srv.close()


@pytest.mark.parametrize("name,m,nb", [("c1", 5, 8), ("c2", 37, 8), ("c2", 1024, 16), ("c5", 1024, 16)])
def test_user_side_of_algorithm_1_is_computed_when_only_U_is_given(name, m, nb):
    """aif_user_precompute with bea_U instead of bea_V: W = Softmax(B U^T / sqrt(d)), V_k = W_f (sum_j W_kj U_j) on the GPU,
    against the oracle; then scoring with the BEA block on, where the item-side weights meet these vectors (step 4).
    The largest sizes the header allows (1024 features, 16 bridges, d up to 256) are included."""
    wl = helpers.MINI[name].with_(name=f"bea_user_{name}", blocks=helpers.ALL_BLOCKS, N=200, L=40, n_bridge=nb, R=1,
                                  lsh_din_norm=synth.NORM_MEAN, simtier_norm=synth.NORM_MEAN, emit_sigmoid=0)
    weights = synth.make_weights(wl)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table)
    dt = orc.F32 if wl.dtype == "f32" else orc.BF16
    rq = synth.make_request(wl, 0)
    U = synth.normal_rows(m, wl.d, 1.0, wl.dtype, 77, m)
    V_want, _ = orc.bea_user(dt, weights["user"]["bridges"], U, weights["user"]["W_f"])
    rq_gpu = dict(rq, bea_U=U)
    del rq_gpu["V"]
    st = srv.precompute(9, srv.upload_request(rq_gpu, B.USER_PROJECTED))
    V_got = srv.ctx.user_state_export_bea(st)
    torch.cuda.synchronize()
    V_got = V_got.float().cpu().numpy().astype(np.float64)
    rtol, atol = (1e-5, 1e-6) if wl.dtype == "f32" else (2.0 ** -8, 1e-4)
    assert np.allclose(V_got, V_want, rtol=rtol, atol=atol), np.abs(V_got - V_want).max()
    # scoring: the oracle gets the vectors the GPU stored (exact inputs), so the usual logit tolerance applies
    stored = V_got.astype(np.float32) if wl.dtype == "f32" else synth.to_bf16_bits(V_got.astype(np.float32))
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    ids = synth.IdSampler(wl).request_ids(0)
    want = oracle.score(table, helpers.projected_request(wl, dict(rq, V=stored)), ids)
    got = srv.score_ids(st, ids)
    assert np.abs(got - want).max() <= (1e-5 if wl.dtype == "f32" else 2e-3)
    # neither V nor U: refused
    rq_none = dict(rq)
    del rq_none["V"]
    with pytest.raises(B.AifError) as e:
        srv.precompute(10, srv.upload_request(rq_none, B.USER_PROJECTED))
    assert e.value.code == B.ERR_ARG
    srv.close()
