"""Parity of the CUDA library (through its C ABI) against the CPU oracle, on the same seeded inputs.

Tolerances (written here, as the benchmark definition states them): |delta logit| <= 1e-5 for the fp32
configuration, <= 2e-3 for bf16 storage with fp32 accumulation; ids, buckets, table rows and signatures are
compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import binding as B
from paper_2511_12934_b200 import build as libbuild
from paper_2511_12934_b200 import serving, synth
from tests import helpers

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-3}


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    B.load_library()


def _setup(wl, path=B.PATH_AUTO, zero_bias=False, **kw):
    weights = synth.make_weights(wl, zero_bias=zero_bias)
    table = synth.make_item_table(wl)
    srv = serving.Server(wl, weights, table, path=path, **kw)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    return weights, table, srv, oracle


def _check_logits(got, want, tol):
    assert got.shape == want.shape
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    err = np.abs(got[ok].astype(np.float64) - want[ok]).max() if ok.any() else 0.0
    assert err <= tol, f"max |delta| = {err:.3e} > {tol}"
    return err


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
@pytest.mark.parametrize("path", [B.PATH_SIMT, B.PATH_AUTO])
def test_scoring_matches_oracle_on_scaled_configs(name, path):
    wl = helpers.MINI[name]
    weights, table, srv, oracle = _setup(wl, path)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r)
        st = srv.precompute(1000 + r, srv.upload_request(rq, B.USER_PROJECTED))
        assert st.request_key == 1000 + r
        want = oracle.score(table, helpers.projected_request(wl, rq), ids)
        got = srv.score_ids(st, ids)
        _check_logits(got, want, TOL[wl.dtype])
        states.append(st), id_lists.append(ids), wants.append(want)
        # mini-batch invariance: one call per chunk gives the same numbers as one call for the request
        chunks = np.concatenate([srv.score_ids(st, ids[s:s + 77]) for s in range(0, len(ids), 77)])
        _check_logits(chunks, want, TOL[wl.dtype])
        if not srv.ctx.get_stats().tensor_path:
            assert np.array_equal(chunks, got)
        # permutation equivariance
        perm = np.random.default_rng(r).permutation(len(ids))
        gp = srv.score_ids(st, ids[perm])
        _check_logits(gp, want[perm], TOL[wl.dtype])
        if not srv.ctx.get_stats().tensor_path:
            assert np.array_equal(gp, got[perm])
    # all requests in one launch
    outs = srv.score_many(states, id_lists)
    for o, w in zip(outs, wants):
        _check_logits(o, w, TOL[wl.dtype])
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("dtype,din_norm,tier_norm", [("f32", synth.NORM_NONE, synth.NORM_NONE),
                                                      ("f32", synth.NORM_MEAN, synth.NORM_MEAN),
                                                      ("bf16", synth.NORM_MEAN, synth.NORM_MEAN)])
def test_all_interaction_blocks(dtype, din_norm, tier_norm):
    base = helpers.MINI["c1"] if dtype == "f32" else helpers.MINI["c2"]
    wl = base.with_(name=f"blocks_{dtype}_{din_norm}", blocks=helpers.ALL_BLOCKS, lsh_din_norm=din_norm,
                    simtier_norm=tier_norm, N=200, L=75, emit_sigmoid=0)
    weights, table, srv, oracle = _setup(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want = oracle.score(table, helpers.projected_request(wl, rq), ids)
    # raw SimTier counts and unnormalised LSH-DIN sums are O(L): scale the absolute tolerance with the logit size
    scale = max(1.0, float(np.abs(want).max()))
    _check_logits(srv.score_ids(st, ids), want, TOL[dtype] * scale)
    srv.close()


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_user_precompute_raw_matches_eqs_1_to_3(name):
    wl = helpers.MINI[name].with_(name=f"raw_{name}", dU=48, L=60, N=150)
    weights, table, srv, oracle = _setup(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(5, srv.upload_request(rq, B.USER_RAW))
    u, S, pu = srv.ctx.user_state_export(st, wl.L)
    torch.cuda.synchronize()
    u_ref, S_ref = oracle.user_state(rq["profile"], rq["seq"])
    W1 = synth.as_f32(weights["mlp"]["W"][0], wl.dtype).astype(np.float64)
    pu_ref = W1[:, :wl.d] @ u_ref + weights["mlp"]["b"][0]
    tol = 1e-5 if wl.dtype == "f32" else 2e-3
    assert np.abs(u.cpu().numpy() - u_ref).max() <= tol
    assert np.abs(S.float().cpu().numpy() - S_ref).max() <= (1e-6 if wl.dtype == "f32" else 2e-3)
    assert np.abs(pu.cpu().numpy() - pu_ref).max() <= tol
    want = oracle.score(table, helpers.raw_request(oracle, rq), ids)
    _check_logits(srv.score_ids(st, ids), want, TOL[wl.dtype])
    # cached state == recomputed state, bit for bit
    st2 = srv.precompute(6, srv.upload_request(rq, B.USER_RAW))
    u2, S2, pu2 = srv.ctx.user_state_export(st2, wl.L)
    torch.cuda.synchronize()
    assert torch.equal(u, u2) and torch.equal(S, S2) and torch.equal(pu, pu2)
    assert np.array_equal(srv.score_ids(st2, ids), srv.score_ids(st, ids))
    srv.close()


def test_refresh_and_gather_are_bit_exact():
    wl = helpers.MINI["c2"].with_(name="refresh", blocks=helpers.ALL_BLOCKS)
    weights, table, srv, oracle = _setup(wl)
    g = np.random.default_rng(3)
    host = {k: v.copy() for k, v in table.items()}
    upd_ids = np.concatenate([g.choice(wl.M, 500, replace=False), [-1, wl.M, 2**31 - 1]]).astype(np.int32)
    new = synth.make_item_table(wl.with_(name="refresh_new"), rows=len(upd_ids))
    for k in ("E", "bea_w", "sig"):
        assert orc.table_refresh(host[k], upd_ids, new[k]) == 3
    srv.refresh_rows(upd_ids, new["E"], new["bea_w"], new["sig"])
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    probe = np.concatenate([upd_ids[:500], g.integers(0, wl.M, 2000)]).astype(np.int32)
    ids_t = torch.from_numpy(probe).cuda()
    out = torch.empty(len(probe), wl.d, dtype=torch.bfloat16, device="cuda")
    srv.ctx.gather_rows(ids_t, out)
    torch.cuda.synchronize()
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, host["E"][probe])
    # scoring after the incremental update sees the new rows, sidecars included
    rq = synth.make_request(wl, 0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    ids = probe[:300]
    want = oracle.score(host, helpers.projected_request(wl, rq), ids)
    _check_logits(srv.score_ids(st, ids), want, TOL["bf16"])
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_bad_ids_edge_sizes_and_errors():
    wl = helpers.MINI["c1"].with_(name="edges", L=1, N=40)
    weights, table, srv, oracle = _setup(wl, max_user_states=2, max_batch_candidates=64)
    rq = synth.make_request(wl, 0)
    dev = srv.upload_request(rq, B.USER_PROJECTED)
    st = srv.precompute(1, dev)
    ids = synth.IdSampler(wl).request_ids(0)
    req = helpers.projected_request(wl, rq)
    # n = 1 and a sequence of length 1
    _check_logits(srv.score_ids(st, ids[:1]), oracle.score(table, req, ids[:1]), TOL["f32"])
    # bad ids -> NaN + status bit, neighbours untouched
    bad = ids.copy()
    bad[3], bad[17] = -5, wl.M
    _check_logits(srv.score_ids(st, bad), oracle.score(table, req, bad), TOL["f32"])
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID and srv.ctx.poll_status() == 0
    # n = 0 is a no-op
    empty = torch.empty(0, dtype=torch.int32, device="cuda")
    srv.ctx.score(st, empty, torch.empty(0, device="cuda"))
    # too many candidates, too long a sequence, arena exhaustion
    with pytest.raises(B.AifError) as e:
        srv.score_ids(st, np.zeros(65, np.int32))
    assert e.value.code == B.ERR_SHAPE
    long_rq = synth.make_request(wl, 0, L=2)
    with pytest.raises(B.AifError) as e:
        srv.precompute(2, srv.upload_request(long_rq, B.USER_PROJECTED))
    assert e.value.code == B.ERR_SHAPE
    st2 = srv.precompute(2, dev)
    with pytest.raises(B.AifError) as e:
        srv.precompute(3, dev)
    assert e.value.code == B.ERR_OOM
    st2.release()
    st3 = srv.precompute(3, dev)
    # reloading weights invalidates cached user states (version consistency)
    srv.ctx.load_weights_host(weights)
    with pytest.raises(B.AifError) as e:
        srv.score_ids(st3, ids)
    assert e.value.code == B.ERR_VERSION
    stats = srv.ctx.get_stats()
    assert stats.model_version == 2 and stats.user_states_high_water == 2 and stats.bad_id_events == 1
    srv.close()


def test_precompute_overlaps_a_simulated_retrieval_phase():
    """The user-side call runs on a side stream while the main stream is busy with 'retrieval'; scoring waits on
    the state's event, so the result is the same as without overlap."""
    wl = helpers.MINI["c3"].with_(name="overlap", R=1)
    weights, table, srv, oracle = _setup(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    dev = srv.upload_request(rq, B.USER_RAW)
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)                      # retrieval stand-in on the main stream
    st = srv.precompute(1, dev)                        # side stream, concurrent
    got = srv.score_ids(st, ids)                       # main stream: waits for both
    want = oracle.score(table, helpers.raw_request(oracle, rq), ids)
    _check_logits(got, want, TOL["bf16"])
    srv.close()


def test_full_size_c1_and_sampled_c2():
    for wl, n_check in ((synth.C1, None), (synth.C2, 1500)):
        weights, table, srv, oracle = _setup(wl, zero_bias=True)
        rq = synth.make_request(wl, 0)
        ids = synth.IdSampler(wl).request_ids(0)
        st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
        got = srv.score_ids(st, ids)
        pick = np.arange(len(ids)) if n_check is None else np.random.default_rng(0).choice(len(ids), n_check, False)
        want = oracle.score(table, helpers.projected_request(wl, rq), ids[pick])
        _check_logits(got[pick], want, TOL[wl.dtype])
        assert np.isfinite(got).all()
        srv.close()


@pytest.mark.parametrize("base,L,s_scale", [("c4", 700, 64.0), ("c4", 700, 1024.0), ("c4", 2500, 1024.0), ("c5", 300, 1024.0),
                                             ("c2", 200, 64.0), ("c2", 200, 1024.0)])
def test_sharp_softmax_exercises_the_running_max_rescaling(base, L, s_scale):
    """Item vectors x32 and sequence rows x64 (exact in bf16) give scores with a standard deviation of about 5: the
    softmax is close to one-hot and the running maximum of the streaming kernels jumps by more than their rescaling
    threshold between key blocks; x1024 gives scores of several hundred (L = 700 and 2500 at d = 128: two softmax warps per
    row, which must agree on every raise; L = 300 at d = 256: one).  With L = 200 the single-launch kernel runs: its first
    softmax attempt subtracts no maximum, which holds at x64 and overflows at x1024, where the kernel must fall back to
    exact row maxima.  Activations are O(1) or more here instead of O(0.05), so the bf16 budget is scaled: bf16
    intermediates of magnitude A carry about 2^-9 A of rounding error."""
    wl = helpers.MINI[base].with_(name="sharp", R=1, N=300, L=L, mini_batch=0)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    table["E"] = synth.to_bf16_bits(synth.bf16_bits_to_f32(table["E"]) * 32.0)
    rq = synth.make_request(wl, 0)
    rq["S"] = synth.to_bf16_bits(synth.bf16_bits_to_f32(rq["S"]) * s_scale)
    srv = serving.Server(wl, weights, table)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want, x = oracle.score(table, helpers.projected_request(wl, rq), ids, return_inputs=True)
    att = x[:, 2 * wl.d:3 * wl.d]
    assert np.abs(att).max() > 1.0                      # the attention really is sharp: outputs near single rows of S
    got = srv.score_ids(st, ids)
    scale = max(1.0, float(np.abs(want).max()))
    _check_logits(got, want, 1e-2 * scale)
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("base,L", [("c2", 700), ("c5", 300)])
def test_softmax_with_and_without_a_running_maximum_in_one_launch(base, L):
    """The attention kernel drops the running maximum for a request whose scores are bounded by 2^+-50 (largest item norm
    x largest sequence-row norm x log2(e) / sqrt(d)).  Four requests in one launch: the workload's own sequence (bound of
    a few units), the sequence scaled to a bound of 45 and of 55 (either side of the switch) and of 600; every tile takes
    its own mode and all must agree with the oracle.  Then a refresh writes one item vector 64 times longer: the table's
    bound only grows, every request falls back to the exact form, and the results stay the same."""
    wl = helpers.MINI[base].with_(name=f"modes_{base}", R=4, N=300, L=L, mini_batch=0)
    weights, table, srv, oracle = _setup(wl, zero_bias=False, max_batch_candidates=wl.R * wl.N)
    E = synth.bf16_bits_to_f32(table["E"])
    e_norm = float(np.sqrt((E.astype(np.float64) ** 2).sum(1)).max())
    k2 = np.log2(np.e) / np.sqrt(wl.d)
    sampler = synth.IdSampler(wl)
    states, id_lists, reqs = [], [], []
    for r, target in enumerate([None, 45.0, 55.0, 600.0]):
        rq = synth.make_request(wl, r)
        if target is not None:
            S = synth.bf16_bits_to_f32(rq["S"]).astype(np.float64)
            k_norm = float(np.sqrt((S ** 2).sum(1)).max())
            rq["S"] = synth.to_bf16_bits((S * (target / (e_norm * k_norm * k2))).astype(np.float32))
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r)), reqs.append(helpers.projected_request(wl, rq))
    wants = [oracle.score(table, reqs[r], id_lists[r]) for r in range(wl.R)]

    def check():
        for o, w in zip(srv.score_many(states, id_lists), wants):
            _check_logits(o, w, 1e-2 * max(1.0, float(np.abs(w).max())))
        _check_logits(srv.score_ids(states[1], id_lists[1]), wants[1], 1e-2 * max(1.0, float(np.abs(wants[1]).max())))
        assert srv.ctx.get_stats().tensor_path == 1 and srv.ctx.poll_status() == 0

    check()
    # a row no candidate uses, 64 times longer than any other
    used = np.unique(np.concatenate(id_lists))
    spare = int(np.setdiff1d(np.arange(table["E"].shape[0]), used)[0])
    row = synth.to_bf16_bits(E[spare:spare + 1] * 64.0 + 1.0)
    srv.refresh_rows(np.array([spare], dtype=np.int32), row)
    check()
    srv.close()


@pytest.mark.parametrize("L", [1, 77, 128, 129, 200, 256, 257])
def test_single_launch_scoring_at_the_sequence_lengths_around_its_key_blocks(L):
    """Launches of at most one tile per SM with sequences of at most 256 items run the whole pass in one kernel (one or
    two key blocks of 128); L = 257 takes the kernel-per-layer path on the same inputs.  Ragged last tiles, a launch of
    several requests, ids outside the table and a zero-length tail of the id array are included."""
    wl = helpers.MINI["c2"].with_(name=f"fused_L{L}", R=2, N=333, L=L, mini_batch=0)
    weights, table, srv, oracle = _setup(wl)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r).copy()
        if r == 1:
            ids[5], ids[200] = -3, table["E"].shape[0]
        st = srv.precompute(7 + r, srv.upload_request(rq, B.USER_PROJECTED))
        want = oracle.score(table, helpers.projected_request(wl, rq), ids)
        _check_logits(srv.score_ids(st, ids), want, TOL["bf16"])
        states.append(st), id_lists.append(ids), wants.append(want)
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    for o, w in zip(srv.score_many(states, id_lists), wants):
        _check_logits(o, w, TOL["bf16"])
    assert srv.ctx.poll_status() == B.STATUS_BAD_ID
    _check_logits(srv.score_ids(states[0], id_lists[0][:1]), wants[0][:1], TOL["bf16"])
    srv.close()


@pytest.mark.parametrize("L", [1, 40, 64, 65, 128, 129, 192, 193, 320, 321])
def test_attention_kernel_at_the_sequence_lengths_around_its_half_blocks(L):
    """d = 128 on the kernel-per-layer path at every length class (a first layer of 256 units is not a shape of the
    single-launch kernel, so short sequences reach the attention kernel too).  Two softmax warps share each candidate row,
    each with 64 of a block's 128 keys: the last block leaves the second warp no key at all (L mod 128 in 1..64), a single
    key (65) or all of them (0), and both must still agree on the block maximum and the row sum.  Two requests in one
    launch, ragged last tiles."""
    wl = helpers.MINI["c2"].with_(name=f"att_L{L}", R=2, N=333, L=L, mini_batch=0, hidden=(256, 256))
    weights, table, srv, oracle = _setup(wl, zero_bias=False)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r)
        states.append(srv.precompute(3 + r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(ids), wants.append(oracle.score(table, helpers.projected_request(wl, rq), ids))
    _check_logits(srv.score_ids(states[0], id_lists[0]), wants[0], TOL["bf16"])
    for o, w in zip(srv.score_many(states, id_lists), wants):
        _check_logits(o, w, TOL["bf16"])
    assert srv.ctx.get_stats().tensor_path == 1
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("base", ["c2", "c5"])
def test_one_launch_over_requests_of_different_sequence_lengths(base):
    """d = 128 and d = 256.  More tiles than SMs on the kernel-per-layer path: every CTA of the attention kernel walks over several tiles, and
    the sequences differ in length from request to request (1 to 321 keys: one to three key blocks, the last one with
    its second half empty, partly filled or full), so consecutive tiles of a CTA have different block counts.  The oracle
    checks a seeded sample of every request, first and last candidate included."""
    Ls = [321, 1, 129, 64, 200, 257]
    wl = helpers.MINI[base].with_(name=f"mixed_L_{base}", R=len(Ls), N=3400, L=max(Ls), mini_batch=0)
    if base == "c2":
        wl = wl.with_(hidden=(256, 256))   # not a shape of the single-launch kernel
    weights, table, srv, oracle = _setup(wl, zero_bias=False, max_batch_candidates=wl.R * wl.N)
    sampler = synth.IdSampler(wl)
    states, id_lists, reqs = [], [], []
    for r, L in enumerate(Ls):
        rq = synth.make_request(wl, r, L=L)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r)), reqs.append(helpers.projected_request(wl, rq))
    outs = srv.score_many(states, id_lists)
    assert srv.ctx.get_stats().tensor_path == 1
    g = np.random.default_rng(23)
    for r in range(wl.R):
        ids = id_lists[r]
        pick = np.unique(np.concatenate([[0, len(ids) - 1], g.choice(len(ids), 38, replace=False)]))
        _check_logits(outs[r][pick], oracle.score(table, reqs[r], ids[pick]), TOL["bf16"])
        assert np.isfinite(outs[r]).all()
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("L", [200, 300])
def test_several_requests_with_mini_batches_in_one_launch(L):
    """Requests of different sizes, each cut into mini-batches of 500 (tiles never straddle a mini-batch), scored in one
    launch: the tile table of the kernel-per-layer path (L = 300) and the request search of the single-launch kernel
    (L = 200) must both place every tile in its request."""
    wl = helpers.MINI["c2"].with_(name=f"batch_mb_{L}", R=4, N=1100, L=L, mini_batch=500, mixed_sizes=(300, 1300))
    weights, table, srv, oracle = _setup(wl)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r)
        states.append(srv.precompute(20 + r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(ids)
        wants.append(oracle.score(table, helpers.projected_request(wl, rq), ids))
    assert len({len(x) for x in id_lists}) > 1
    for o, w in zip(srv.score_many(states, id_lists), wants):
        _check_logits(o, w, TOL["bf16"])
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("L", [200, 300])
def test_a_launch_with_empty_requests_among_the_others(L):
    """Requests without candidates at the start, in the middle and at the end of a batch: their tiles do not exist, and
    every existing tile must still find its own request (single-launch kernel at L = 200, tile table at L = 300)."""
    wl = helpers.MINI["c2"].with_(name=f"empty_req_{L}", R=5, N=260, L=L, mini_batch=0)
    weights, table, srv, oracle = _setup(wl)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r) if r in (1, 3) else np.zeros(0, dtype=np.int32)
        states.append(srv.precompute(30 + r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(ids)
        wants.append(oracle.score(table, helpers.projected_request(wl, rq), ids) if len(ids) else np.zeros(0))
    outs = srv.score_many(states, id_lists)
    for o, w in zip(outs, wants):
        assert len(o) == len(w)
        if len(w):
            _check_logits(o, w, TOL["bf16"])
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("H2,F,dc,Bk,mode,sig", [(64, 2, 32, 1024, synth.BUCKET_HASH, 0), (128, 8, 8, 1000, synth.BUCKET_HASH, 1),
                                                  (192, 12, 16, 1024, synth.BUCKET_MOD, 0), (256, 8, 64, 37, synth.BUCKET_MOD, 1),
                                                  (256, 24, 16, 512, synth.BUCKET_HASH, 0)])
def test_single_launch_scoring_over_the_shapes_it_accepts(H2, F, dc, Bk, mode, sig):
    """Second-layer widths 64..256, one to eight cross-feature chunks of 64 columns, cross embeddings of 8..64 columns
    (eight fields to one field per chunk), bucket counts that are and are not powers of two, both bucket functions, with and
    without the final sigmoid; non-zero biases, which this kernel adds on the tensor cores."""
    wl = helpers.MINI["c2"].with_(name=f"fused_{H2}_{F}_{dc}", R=1, N=300, L=150, mini_batch=0, hidden=(512, H2), F=F, dc=dc,
                                  B=Bk, bucket_mode=mode, emit_sigmoid=sig)
    weights, table, srv, oracle = _setup(wl, zero_bias=False)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(3, srv.upload_request(rq, B.USER_PROJECTED))
    want = oracle.score(table, helpers.projected_request(wl, rq), ids)
    _check_logits(srv.score_ids(st, ids), want, TOL["bf16"])
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("hidden", [(256, 48), (192, 16), (128, 64, 80), (512, 112)])
def test_last_hidden_width_that_is_not_a_multiple_of_32(hidden):
    """The kernel-per-layer path reads an accumulator 32 columns at a time; the last width only has to be a multiple of
    16, so its last read is half used and the other half (columns no product wrote) must not reach the logit."""
    wl = helpers.MINI["c2"].with_(name=f"h_{'_'.join(map(str, hidden))}", R=2, N=300, L=70, mini_batch=0, hidden=hidden)
    weights, table, srv, oracle = _setup(wl, zero_bias=False)
    sampler = synth.IdSampler(wl)
    for r in range(wl.R):          # the second call finds whatever the first left in tensor and shared memory
        rq = synth.make_request(wl, r)
        ids = sampler.request_ids(r)
        st = srv.precompute(3 + r, srv.upload_request(rq, B.USER_PROJECTED))
        _check_logits(srv.score_ids(st, ids), oracle.score(table, helpers.projected_request(wl, rq), ids), TOL["bf16"])
    assert srv.ctx.get_stats().tensor_path == 1
    assert srv.ctx.poll_status() == 0
    srv.close()


@pytest.mark.parametrize("name", ["c3", "c4", "c5", "c5b"])
def test_full_size_batches_on_sampled_candidates(name):
    """The multi-request shapes at their full sizes, scored in one aif_score_batch call exactly as the benchmark
    launches them; the oracle checks a seeded sample of candidates of a few requests (first, middle, last)."""
    wl = synth.SHORT[name]
    weights, table, srv, oracle = _setup(wl, zero_bias=False)
    sampler = synth.IdSampler(wl)
    states, id_lists, reqs = [], [], {}
    check = sorted({0, wl.R // 2, wl.R - 1})
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r))
        if r in check:
            reqs[r] = helpers.projected_request(wl, rq)
    outs = srv.score_many(states, id_lists)
    assert srv.ctx.get_stats().tensor_path == 1
    g = np.random.default_rng(11)
    worst = 0.0
    for r in check:
        ids = id_lists[r]
        # the sample always contains the request's first and last candidate (tile edges)
        pick = np.unique(np.concatenate([[0, len(ids) - 1], g.choice(len(ids), 48, replace=False)]))
        want = oracle.score(table, reqs[r], ids[pick])
        worst = max(worst, _check_logits(outs[r][pick], want, TOL["bf16"]))
    for o in outs:
        assert np.isfinite(o).all()
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_a_wait_that_runs_out_sets_the_timeout_bit_and_leaves_the_context_usable():
    """Failure detection without a fault: the device-side waits are bounded.  A kernel whose wait nobody satisfies gives
    up after its limit, reports AIF_STATUS_TIMEOUT through the status word and returns; scoring afterwards is intact."""
    wl = helpers.MINI["c2"].with_(name="timeout", N=300)
    weights, table, srv, oracle = _setup(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want = oracle.score(table, helpers.projected_request(wl, rq), ids)
    _check_logits(srv.score_ids(st, ids), want, TOL["bf16"])
    assert srv.ctx.poll_status() == 0
    srv.ctx.selftest_bounded_wait(2_000_000)            # about a millisecond
    assert srv.ctx.poll_status() == B.STATUS_TIMEOUT
    assert srv.ctx.get_stats().timeout_events == 1
    assert srv.ctx.poll_status() == 0                   # read and cleared
    _check_logits(srv.score_ids(st, ids), want, TOL["bf16"])
    with pytest.raises(B.AifError) as e:
        srv.ctx.selftest_bounded_wait(0)
    assert e.value.code == B.ERR_ARG
    srv.close()


def test_score_host_with_pinned_and_with_pageable_buffers():
    """aif_score_host takes the zero-copy route for pinned (mapped) buffers and the staged route for pageable ones;
    both give the device-buffer result bit for bit."""
    wl = helpers.MINI["c2"].with_(name="hostbuf", N=777)
    weights, table, srv, oracle = _setup(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    ref = srv.score_ids(st, ids)
    for pinned in (True, False):
        h_ids = torch.from_numpy(ids.copy())
        h_out = torch.full((len(ids),), float("nan"), dtype=torch.float32)
        if pinned:
            h_ids, h_out = h_ids.pin_memory(), h_out.pin_memory()
        srv.ctx.score_host(st, h_ids, h_out)
        assert np.array_equal(h_out.numpy(), ref)
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_score_batch_host_gives_the_device_buffer_result():
    """aif_score_batch_host (host ids in, host logits out, several requests in one launch) equals aif_score_batch on
    device buffers bit for bit, with page-locked and with pageable buffers, and matches the oracle."""
    wl = helpers.MINI["c3"].with_(name="hostbatch", R=3, N=333)
    weights, table, srv, oracle = _setup(wl)
    sampler = synth.IdSampler(wl)
    states, id_lists, wants = [], [], []
    for r in range(wl.R):
        rq = synth.make_request(wl, r)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r, 333 - 100 * r))
        wants.append(oracle.score(table, helpers.projected_request(wl, rq), id_lists[-1]))
    ref = np.concatenate(srv.score_many(states, id_lists))
    offs = np.zeros(wl.R + 1, dtype=np.int64)
    offs[1:] = np.cumsum([len(x) for x in id_lists])
    for pinned in (True, False):
        h_ids = torch.from_numpy(np.concatenate(id_lists))
        h_out = torch.full((int(offs[-1]),), float("nan"), dtype=torch.float32)
        if pinned:
            h_ids, h_out = h_ids.pin_memory(), h_out.pin_memory()
        srv.ctx.score_batch_host(states, h_ids, offs, h_out)
        assert np.array_equal(h_out.numpy(), ref)
    _check_logits(ref, np.concatenate(wants), TOL["bf16"])
    with pytest.raises(B.AifError) as e:     # more candidates than the context was sized for
        big = torch.zeros(wl.R * wl.N + 1, dtype=torch.int32)
        srv.ctx.score_batch_host(states[:1], big, [0, len(big)], torch.zeros(len(big)))
    assert e.value.code == B.ERR_SHAPE
    assert srv.ctx.poll_status() == 0
    srv.close()


def test_versioned_table_full_refresh_is_published_as_a_whole():
    """versioned_table: a scoring call made before a full refresh keeps reading the old copy even though it runs after the
    refresh has written (it sits behind a busy main stream while the refresh runs on a side stream); a call made after
    the refresh reads the new copy.  A full refresh of fewer rows than the table carries the rest over; incremental
    refreshes and the gather see the live copy; a second full refresh swaps back."""
    wl = helpers.MINI["c2"].with_(name="versioned", N=600, blocks=helpers.ALL_BLOCKS)
    weights = synth.make_weights(wl, zero_bias=False)
    tab_a = synth.make_item_table(wl)
    tab_b = synth.make_item_table(wl.with_(name="versioned_b"))
    srv = serving.Server(wl, weights, tab_a, versioned_table=1)
    oracle = helpers.make_oracle(wl, weights, M=tab_a["E"].shape[0])
    rq = synth.make_request(wl, 0)
    req = helpers.projected_request(wl, rq)
    ids = synth.IdSampler(wl).request_ids(0)
    st = srv.precompute(1, srv.upload_request(rq, B.USER_PROJECTED))
    want_a, want_b = oracle.score(tab_a, req, ids), oracle.score(tab_b, req, ids)
    assert np.abs(want_a - want_b).max() > 0.01
    _check_logits(srv.score_ids(st, ids), want_a, TOL["bf16"])
    ids_t = torch.from_numpy(ids).cuda()
    out_old = torch.empty(len(ids), dtype=torch.float32, device="cuda")
    out_new = torch.empty(len(ids), dtype=torch.float32, device="cuda")
    dt = srv.dt
    E_b, bw_b = B.to_device(tab_b["E"], dt), B.to_device(tab_b["bea_w"], dt)
    sg_b = torch.from_numpy(np.ascontiguousarray(tab_b["sig"])).cuda()
    torch.cuda.synchronize()
    torch.cuda._sleep(40_000_000)                                  # the main stream is busy for some 20 ms
    srv.ctx.score(st, ids_t, out_old)                              # made before the refresh: the old copy
    with torch.cuda.stream(srv.side):
        srv.ctx.item_nearline_refresh(None, E_b, bw_b, sg_b, stream=srv.side)   # runs at once, beside the sleeping main stream
    srv.ctx.score(st, ids_t, out_new)                              # made after it: the new copy, once it is complete
    torch.cuda.synchronize()
    _check_logits(out_old.cpu().numpy(), want_a, TOL["bf16"])
    _check_logits(out_new.cpu().numpy(), want_b, TOL["bf16"])
    # a full refresh of the first half only: the second half is carried over from the live copy (table B)
    half = tab_a["E"].shape[0] // 2
    srv.ctx.item_nearline_refresh(None, B.to_device(tab_a["E"][:half], dt), B.to_device(tab_a["bea_w"][:half], dt),
                                  torch.from_numpy(np.ascontiguousarray(tab_a["sig"][:half])).cuda())
    mixed = {k: np.concatenate([tab_a[k][:half], tab_b[k][half:]]) for k in ("E", "bea_w", "sig")}
    _check_logits(srv.score_ids(st, ids), oracle.score(mixed, req, ids), TOL["bf16"])
    # incremental refresh and gather address the live copy
    upd = np.array([int(ids[0]), int(ids[5])], dtype=np.int32)
    for k in ("E", "bea_w", "sig"):
        mixed[k] = mixed[k].copy()
        mixed[k][upd] = tab_b[k][upd] if upd[0] < half else tab_a[k][upd]
    srv.refresh_rows(upd, mixed["E"][upd], mixed["bea_w"][upd], mixed["sig"][upd])
    _check_logits(srv.score_ids(st, ids), oracle.score(mixed, req, ids), TOL["bf16"])
    got = torch.empty(len(ids), wl.d, dtype=torch.bfloat16, device="cuda")
    srv.ctx.gather_rows(ids_t, got)
    torch.cuda.synchronize()
    assert np.array_equal(got.view(torch.int16).cpu().numpy().view(np.uint16), mixed["E"][ids])
    assert srv.ctx.poll_status() == 0 and srv.ctx.get_stats().table_version == 4
    srv.close()


@pytest.mark.parametrize("kind", ["fused", "chain", "blocks", "categories", "simt"])
def test_nothing_is_written_outside_the_logits(kind):
    """Canary words on both sides of the logit array (which therefore starts on an odd 4-byte boundary) stay untouched by
    every scoring path: the single-launch kernel, the kernel-per-layer chain, the chain with all blocks, grouped
    candidates, and the CUDA-core kernel; ragged last tiles and a launch of several requests included."""
    base = {"fused": helpers.MINI["c2"].with_(L=150), "chain": helpers.MINI["c2"].with_(L=300),
            "blocks": helpers.MINI["c2"].with_(L=300, blocks=helpers.ALL_BLOCKS),
            "categories": helpers.MINI["c2"].with_(L=300, blocks=helpers.ALL_BLOCKS, n_categories=6),
            "simt": helpers.MINI["c1"]}[kind]
    wl = base.with_(name=f"canary_{kind}", R=3, N=333, mini_batch=0)
    weights, table, srv, oracle = _setup(wl)
    sampler = synth.IdSampler(wl)
    states, id_lists = [], []
    for r in range(wl.R):
        states.append(srv.precompute(r, srv.upload_request(synth.make_request(wl, r), B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r, 333 - 101 * r))
    guard, sentinel = 67, -12345.5
    for ids_l, sts in (([id_lists[0]], [states[0]]), (id_lists, states)):
        n = sum(len(x) for x in ids_l)
        buf = torch.full((n + 2 * guard,), sentinel, dtype=torch.float32, device="cuda")
        ids_t = torch.from_numpy(np.concatenate(ids_l)).cuda()
        offs = np.concatenate([[0], np.cumsum([len(x) for x in ids_l])])
        if len(sts) == 1:
            srv.ctx.score(sts[0], ids_t, buf[guard:guard + n])
        else:
            srv.ctx.score_batch(sts, ids_t, offs, buf[guard:guard + n])
        torch.cuda.synchronize()
        h = buf.cpu().numpy()
        assert (h[:guard] == sentinel).all() and (h[guard + n:] == sentinel).all()
        assert np.isfinite(h[guard:guard + n]).all() and not (h[guard:guard + n] == sentinel).any()
    assert srv.ctx.poll_status() == 0
    srv.close()
