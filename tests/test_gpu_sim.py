"""Category sub-sequences (Section 3.3, SIM-hard) on the GPU against the CPU oracle: the user side groups the sequence by
category, the real-time phase groups the candidates by (request, category), and the attention / LSH kernels see only the
candidate's category's sub-sequence.  |delta logit| <= 2e-3 (bf16 storage, fp32 accumulation)."""
import numpy as np
import pytest
import torch

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import binding as B
from paper_2511_12934_b200 import build as libbuild
from paper_2511_12934_b200 import serving, synth
from tests import helpers

pytestmark = pytest.mark.gpu

TOL = 2e-3
LSH = synth.BLK_LSH_DIN | synth.BLK_SIMTIER


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    B.load_library()


def _check(got, want, tol=TOL):
    assert got.shape == want.shape
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    err = np.abs(got[ok].astype(np.float64) - want[ok]).max() if ok.any() else 0.0
    assert err <= tol, f"max |delta| = {err:.3e} > {tol}"


@pytest.mark.parametrize("base,blocks,n_cat", [("c2", synth.BLK_ATT | synth.BLK_CROSS, 7), ("c2", synth.BLK_ATT | synth.BLK_CROSS | LSH, 100),
                                               ("c2", helpers.ALL_BLOCKS, 1), ("c2", synth.BLK_CROSS | LSH, 13),
                                               ("c5", helpers.ALL_BLOCKS, 20), ("c5", synth.BLK_ATT | synth.BLK_CROSS, 3)])
def test_sub_sequences_by_category_in_one_launch_and_request_by_request(base, blocks, n_cat):
    """Four requests with sequences of 1 to 1500 items and 1 to 2100 candidates.  With 100 categories most sub-sequences of
    the short sequences are empty (zero rows by the oracle's reading) and most groups hold a handful of candidates; with
    one category the grouped path must reproduce the whole-sequence result."""
    Ls = [1500, 1, 130, 700]
    sizes = [2100, 333, 1, 900]
    wl = helpers.MINI[base].with_(name=f"sim_{base}_{blocks}_{n_cat}", R=len(Ls), N=max(sizes), L=max(Ls), mini_batch=0, blocks=blocks,
                                  n_categories=n_cat)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR, max_batch_candidates=sum(sizes))
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    sampler = synth.IdSampler(wl)
    states, id_lists, reqs = [], [], []
    for r, (L, n) in enumerate(zip(Ls, sizes)):
        rq = synth.make_request(wl, r, L=L)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r, n)), reqs.append(helpers.projected_request(wl, rq))
    wants = [oracle.score(table, reqs[r], id_lists[r]) for r in range(wl.R)]
    for o, w in zip(srv.score_many(states, id_lists), wants):
        _check(o, w)
    for r in (0, 2, 3):
        _check(srv.score_ids(states[r], id_lists[r]), wants[r])
    # ids outside the table among the candidates: NaN, status bit, neighbours untouched
    ids = id_lists[3].copy()
    ids[0], ids[500] = -7, table["E"].shape[0]
    _check(srv.score_ids(states[3], ids), oracle.score(table, reqs[3], ids))
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    if n_cat == 1:
        plain = wl.with_(n_categories=0)
        po = helpers.make_oracle(plain, weights, M=table["E"].shape[0])
        assert np.array_equal(po.score(table, reqs[0], id_lists[0]), wants[0])
    srv.close()


def test_category_of_a_sequence_item_outside_the_range_drops_the_item():
    wl = helpers.MINI["c2"].with_(name="sim_badcat", R=1, N=400, L=300, mini_batch=0, blocks=synth.BLK_ATT | synth.BLK_CROSS | LSH,
                                  n_categories=5)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    rq = synth.make_request(wl, 0)
    rq["seq_cat"][[3, 77, 299]] = [-1, 5, 1 << 20]        # never equal to a candidate's category: in no sub-sequence
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    _check(srv.score_ids(st, ids), oracle.score(table, helpers.projected_request(wl, rq), ids))
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    # the same slot again with a shorter sequence: nothing of the longer one may be left in the grouped rows
    st.release()
    rq2 = synth.make_request(wl, 1, L=40)
    st2 = srv.precompute(2, srv.upload_request(rq2, B.USER_PROJECTED))
    _check(srv.score_ids(st2, ids), oracle.score(table, helpers.projected_request(wl, rq2), ids))
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_raw_user_state_with_categories():
    """eqs. 1-3 run on the sequence in its own order; the grouped copy is made from the projected rows they produce."""
    wl = helpers.MINI["c2"].with_(name="sim_raw", R=1, N=300, L=260, mini_batch=0, n_categories=9)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_RAW))
    _check(srv.score_ids(st, ids), oracle.score(table, helpers.raw_request(oracle, rq), ids))
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_categories_need_the_tensor_core_kernels():
    wl = helpers.MINI["c1"].with_(name="sim_f32", n_categories=4)
    with pytest.raises(B.AifError) as e:
        serving.Server(wl, synth.make_weights(wl), synth.make_item_table(wl))
    assert e.value.code == B.ERR_SHAPE


@pytest.mark.parametrize("n_cat", [0, 100])
def test_lsh_only_scoring_against_a_sequence_of_1e5_items(n_cat):
    """The long-term sequence of Section 3.3 / 4.2 (length ~10^5) with the LSH blocks in place of the dense attention: the
    whole sequence (n_cat = 0: 782 key blocks per tile) and its category sub-sequences (about 1000 items each)."""
    wl = synth.C4.with_(name=f"lsh_1e5_{n_cat}", R=1, N=700, M=50_000, L=100_000, blocks=synth.BLK_CROSS | LSH, n_categories=n_cat)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    got = srv.score_ids(st, ids)
    pick = np.unique(np.concatenate([[0, 127, 128, len(ids) - 1], np.random.default_rng(3).choice(len(ids), 60, replace=False)]))
    _check(got[pick], oracle.score(table, helpers.projected_request(wl, rq), ids[pick]))
    assert np.isfinite(got).all() and srv.ctx.poll_status() == 0
    srv.close()
