"""Parity of the paper's approximation blocks (Algorithm 1 step 4; eqs. 6-9) and of the raw user-side path (eqs. 1-3)
on the launch shapes that serving uses: several requests in one launch, mini-batches, more tiles than the GPU has SMs,
d = 128 and d = 256, the long-sequence shape at full size.  Every comparison is element by element against the CPU
oracle, |delta logit| <= 2e-3 (bf16 storage, fp32 accumulation)."""
import numpy as np
import pytest
import torch

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
    return err


def _edges(n, mb, g, extra):
    """Positions worth checking in a request of n candidates: both ends, the rows on either side of every tile and
    mini-batch boundary that exists, and a seeded sample of the rest."""
    pts = {0, n - 1}
    step = mb if mb > 0 else n
    for b0 in range(0, n, step):
        b1 = min(n, b0 + step)
        pts.update((b0, b1 - 1))
        for t in range(b0, b1, 128):
            pts.update((t, max(b0, t - 1)))
    if n > extra:
        pts.update(int(x) for x in g.choice(n, extra, replace=False))
    else:
        pts.update(range(n))
    return np.array(sorted(p for p in pts if 0 <= p < n), dtype=np.int64)


@pytest.mark.parametrize("base,blocks", [("c2", helpers.ALL_BLOCKS), ("c5", helpers.ALL_BLOCKS),
                                         ("c2", synth.BLK_CROSS | LSH), ("c2", synth.BLK_ATT | synth.BLK_SIMTIER),
                                         ("c2", synth.BLK_CROSS | synth.BLK_LSH_DIN | synth.BLK_BEA)])
def test_blocks_in_one_launch_over_requests_of_different_sizes_and_lengths(base, blocks):
    """Six requests of 1 to 5200 candidates with sequences of 1 to 321 items, cut into mini-batches of 500, scored by one
    aif_score_batch call: 150 tiles, more than the GPU has SMs.  d = 128 with two hidden layers and d = 256 with three;
    all blocks on, and subsets of them (dense attention off, one LSH block alone)."""
    Ls = [321, 1, 129, 64, 200, 257]
    sizes = [5000, 300, 4100, 1, 3777, 5200]
    wl = helpers.MINI[base].with_(name=f"blocks_batch_{base}_{blocks}", R=len(Ls), N=max(sizes), L=max(Ls), mini_batch=500,
                                  blocks=blocks)
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
    outs = srv.score_many(states, id_lists)
    g = np.random.default_rng(5)
    for r in range(wl.R):
        ids = id_lists[r]
        pick = _edges(len(ids), wl.mini_batch, g, 400 if base == "c2" else 120)
        _check(outs[r][pick], oracle.score(table, reqs[r], ids[pick]))
        assert np.isfinite(outs[r]).all()
    # the same requests one by one (one launch each, mini-batches inside)
    for r in (1, 3, 4):
        got = srv.score_ids(states[r], id_lists[r])
        pick = _edges(len(got), wl.mini_batch, g, 100)
        _check(got[pick], oracle.score(table, reqs[r], id_lists[r][pick]))
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_small_mini_batches_need_more_tiles_than_candidates_over_128():
    """Mini-batches of 100: every tile holds at most 100 candidates, so a launch has about 28 % more tiles than
    candidates / 128.  The tile table must hold them all, and every tile must land in its own request."""
    sizes = [2500, 730, 1, 99, 100, 101, 3100]
    wl = helpers.MINI["c2"].with_(name="small_mb", R=len(sizes), N=max(sizes), L=300, mini_batch=100)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR, max_batch_candidates=sum(sizes))
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r, n in enumerate(sizes):
        rq = synth.make_request(wl, r)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r, n))
        wants.append(oracle.score(table, helpers.projected_request(wl, rq), id_lists[-1]))
    for o, w in zip(srv.score_many(states, id_lists), wants):
        _check(o, w)
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("blocks", [helpers.ALL_BLOCKS, synth.BLK_CROSS | LSH])
def test_long_sequence_shape_at_full_size_with_the_lsh_blocks(blocks):
    """16 requests x 10^4 candidates against sequences of 10^4 items, one aif_score_batch call as the benchmark launches
    it, with LSH-DIN and SimTier on (and, in the first variant, the dense attention and BEA as well).  The oracle checks
    a seeded sample of the first, a middle and the last request, first and last candidate included."""
    wl = synth.C4.with_(name=f"c4_lsh_{blocks}", blocks=blocks)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    sampler = synth.IdSampler(wl)
    states, id_lists, reqs = [], [], {}
    check = (0, wl.R // 2, wl.R - 1)
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r))
        if r in check:
            reqs[r] = helpers.projected_request(wl, rq)
    outs = srv.score_many(states, id_lists)
    g = np.random.default_rng(17)
    for r in check:
        ids = id_lists[r]
        pick = np.unique(np.concatenate([[0, 127, 128, len(ids) - 1], g.choice(len(ids), 44, replace=False)]))
        _check(outs[r][pick], oracle.score(table, reqs[r], ids[pick]))
    for o in outs:
        assert np.isfinite(o).all()
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("base,L", [("c4", 10_000), ("c5", 500), ("c5", 1100), ("c2", 1000), ("c2", 1024)])
def test_raw_user_precompute_at_long_sequences(base, L):
    """eqs. 1-3 from raw embeddings at the lengths where the tuned path is live: the self-attention rows come from the
    tensor-core attention kernel over many tiles, eq. 3 is merged from 256 key slices.  u, p_u and every row of the
    projected sequence are compared with the oracle's orc_user_state, then a request is scored on the cached state."""
    wl = synth.SHORT[base].with_(name=f"raw_long_{base}", R=1, N=400, M=20_000, L=L)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    rq = synth.make_request(wl, 0)
    st = srv.precompute(5, srv.upload_request(rq, B.USER_RAW))
    u, S, pu = srv.ctx.user_state_export(st, wl.L)
    torch.cuda.synchronize()
    u_ref, S_ref = oracle.user_state(rq["profile"], rq["seq"])
    W1 = synth.as_f32(weights["mlp"]["W"][0], wl.dtype).astype(np.float64)
    pu_ref = W1[:, :wl.d] @ u_ref + weights["mlp"]["b"][0]
    assert np.abs(S.float().cpu().numpy() - S_ref).max() <= TOL
    assert np.abs(u.cpu().numpy() - u_ref).max() <= TOL
    assert np.abs(pu.cpu().numpy() - pu_ref).max() <= TOL
    ids = synth.IdSampler(wl).request_ids(0)
    pick = np.arange(0, len(ids), 4 if L > 2000 else 1)
    want = oracle.score(table, {"u": u_ref, "S": S_ref, "T": rq["T"]}, ids[pick])
    _check(srv.score_ids(st, ids)[pick], want)
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("base,n_tiers,din_norm,tier_norm,blocks", [
    ("c2", 8, synth.NORM_MEAN, synth.NORM_MEAN, helpers.ALL_BLOCKS),
    ("c2", 16, synth.NORM_MEAN, synth.NORM_MEAN, synth.BLK_CROSS | LSH),
    ("c2", 5, synth.NORM_NONE, synth.NORM_NONE, synth.BLK_ATT | synth.BLK_CROSS | LSH),
    ("c2", 1, synth.NORM_MEAN, synth.NORM_NONE, synth.BLK_SIMTIER),
    ("c2", 3, synth.NORM_MEAN, synth.NORM_MEAN, synth.BLK_CROSS | synth.BLK_LSH_DIN),
    ("c5", 16, synth.NORM_MEAN, synth.NORM_MEAN, synth.BLK_CROSS | LSH),
    ("c5", 7, synth.NORM_NONE, synth.NORM_MEAN, helpers.ALL_BLOCKS)])
def test_lsh_blocks_run_on_the_tensor_cores_for_every_tier_count_and_norm(base, n_tiers, din_norm, tier_norm, blocks):
    """The LSH similarity, LSH-DIN and SimTier kernel (signature products in fp8, counts times S in bf16): tier counts 1 to
    16 (tier edges that do and do not divide d'), raw and mean-normalised outputs, either block alone, sequence lengths that
    leave the last key block nearly empty, half full and full, identical signatures (every match count = d', the closed
    last tier) and complementary ones (0 matches).  The kernel list of the call must name the tensor-core kernel."""
    exact = din_norm == synth.NORM_MEAN and tier_norm == synth.NORM_MEAN
    # raw sums and counts (eq. 8 and eq. 9 as printed) grow with the sequence: kept to lengths whose counts bf16 still holds
    # exactly (<= 256), since the MLP input is stored in bf16
    Ls = [1, 63, 64, 65, 127, 128, 129, 700 if exact else 256]
    wl = helpers.MINI[base].with_(name=f"lsh_tc_{base}_{n_tiers}", R=len(Ls), N=300, L=max(Ls), mini_batch=0, blocks=blocks,
                                  n_tiers=n_tiers, lsh_din_norm=din_norm, simtier_norm=tier_norm)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    sampler = synth.IdSampler(wl)
    id_lists = [sampler.request_ids(r) for r in range(wl.R)]
    rqs = [synth.make_request(wl, r, L=L) for r, L in enumerate(Ls)]
    # request 3: every sequence item carries the signature of the request's first candidate, request 4 its complement
    rqs[3]["sig_seq"][:] = table["sig"][id_lists[3][0]]
    rqs[4]["sig_seq"][:] = ~table["sig"][id_lists[4][0]]
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    states = [srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)) for r, rq in enumerate(rqs)]
    srv.ctx.set_kernel_timing(True)
    outs = srv.score_many(states, id_lists)
    assert "lsh" in srv.ctx.get_kernel_timing()
    srv.ctx.set_kernel_timing(False)
    # With mean-normalised outputs every MLP input is below 1 and the tolerance is the plain 2e-3.  Raw sums and counts are
    # inputs of magnitude A >> 1 that the kernel chain stores in bf16 (relative rounding 2^-9), and so are the hidden
    # activations they produce: the tolerance scales with A.  That only checks the plumbing of the unnormalised option; the
    # counts and sums themselves are checked by the normalised cases, which differ by one multiplication.
    def tol_for(x):
        return TOL * (1.0 if exact else max(1.0, float(np.nanmax(np.abs(x)))))

    for r in range(wl.R):
        want, x = oracle.score(table, helpers.projected_request(wl, rqs[r]), id_lists[r], return_inputs=True)
        _check(outs[r], want, tol_for(x))
    # one request alone, with ids outside the table: NaN logits, status bit, neighbours untouched
    ids = id_lists[7].copy()
    ids[3], ids[130] = -1, table["E"].shape[0]
    want, x = oracle.score(table, helpers.projected_request(wl, rqs[7]), ids, return_inputs=True)
    _check(srv.score_ids(states[7], ids), want, tol_for(x))
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    srv.close()
