"""Pins of the CPU oracle against what the paper and the mathematics fix: printed examples, closed forms,
special cases, invariants and brute force on tiny inputs.  No GPU, no CUDA library."""
import math
import os

import numpy as np
import pytest

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import synth
from tests import helpers


# ------------------------------------------------------------------------------------------------
# LSH: packing, popcount table, similarity (Section 4.2, eqs. 5-7)
# ------------------------------------------------------------------------------------------------
def test_packing_matches_printed_example(golden_dir):
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "lsh_packing_example.txt")) if ln[0] != "#"]
    for bitstr, val in rows:
        bits = np.array([int(c) for c in bitstr], dtype=np.uint8)
        assert orc.pack_bits(bits)[0] == int(val)
        assert orc.popcount_lut(int(val)) == bitstr.count("1") == 4


def test_packing_all_bytes_is_msb_first():
    for v in range(256):
        bits = np.array([(v >> (7 - k)) & 1 for k in range(8)], dtype=np.uint8)
        assert orc.pack_bits(bits)[0] == v
    bits = np.random.default_rng(0).integers(0, 2, 128, dtype=np.uint8)
    assert np.array_equal(orc.pack_bits(bits), np.packbits(bits, bitorder="big"))


def test_popcount_table_exhaustive():
    for v in range(256):
        assert orc.popcount_lut(v) == bin(v).count("1")


def test_lsh_matches_against_unpacked_bit_loop():
    g = np.random.default_rng(1)
    for nbits in (8, 64, 128, 256):
        for _ in range(20):
            a = g.integers(0, 2, nbits, dtype=np.uint8)
            b = g.integers(0, 2, nbits, dtype=np.uint8)
            brute = sum(1 for k in range(nbits) if a[k] == b[k])   # XNOR, bit by bit, on unpacked bits
            pa, pb = np.packbits(a), np.packbits(b)
            assert orc.lsh_matches(pa, pb, via_lut=True) == brute
            assert orc.lsh_matches(pa, pb, via_lut=False) == brute
            assert orc.lsh_matches(pb, pa) == brute                 # symmetric
            assert orc.lsh_matches(pa, pa) == nbits                 # sim(x, x) = 1
            assert orc.lsh_matches(pa, ~pa) == 0                    # sim(x, not x) = 0


def test_lsh_similarity_matrix_values_are_multiples_of_one_over_dbits():
    g = np.random.default_rng(2)
    a = g.integers(0, 256, (5, 16), dtype=np.uint8)
    s = g.integers(0, 256, (7, 16), dtype=np.uint8)
    sim = orc.lsh_similarity(a, s, 128)
    assert sim.shape == (5, 7)
    k = sim * 128
    assert np.array_equal(k, np.round(k)) and k.min() >= 0 and k.max() <= 128
    for i in range(5):
        for j in range(7):
            assert k[i, j] == orc.lsh_matches(a[i], s[j])


def test_lsh_hash_sign_convention_and_collision_probability():
    g = np.random.default_rng(3)
    d, dbits = 32, 4096
    W = g.standard_normal((dbits, d))
    assert orc.lsh_hash_bits(np.zeros(d), W).sum() == 0          # Sign(0) = 0 -> bit 0
    m = g.standard_normal(d)
    b = orc.lsh_hash_bits(m, W)
    assert np.array_equal(b, orc.lsh_hash_bits(3.5 * m, W))       # positive scaling keeps every bit
    assert np.array_equal(1 - b, orc.lsh_hash_bits(-m, W))        # negation flips every bit
    assert np.array_equal(b, (W @ m > 0).astype(np.uint8))
    # sign random projections: P[bits agree] = 1 - theta / pi
    for theta in (0.2, 1.0, 2.5):
        e1 = np.zeros(d); e1[0] = 1.0
        e2 = np.zeros(d); e2[0], e2[1] = math.cos(theta), math.sin(theta)
        agree = np.mean(orc.lsh_hash_bits(e1, W) == orc.lsh_hash_bits(e2, W))
        assert abs(agree - (1 - theta / math.pi)) < 4 * math.sqrt(0.25 / dbits)


def test_table4_complexity_bookkeeping(golden_dir):
    # d' bits are stored as d'/8 uint8 lanes: the oracle compares dbits/8 bytes per pair, 8x fewer than d.
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "lsh_complexity_table4.txt")) if ln[0] != "#"]
    for _, cost, red in rows:
        assert abs(100.0 * (1 - float(cost) / 16.0) - float(red)) < 1e-9
    d_lsh_lanes = 128 // 8
    assert (128 + 128) / d_lsh_lanes == 16


# ------------------------------------------------------------------------------------------------
# SimTier and LSH-DIN (eqs. 8-9)
# ------------------------------------------------------------------------------------------------
def test_tier_edges():
    for dbits, T in ((128, 8), (64, 8), (256, 8), (128, 5), (64, 3)):
        assert orc.tier_of(0, dbits, T) == 0
        assert orc.tier_of(dbits, dbits, T) == T - 1          # sim = 1 falls in the last (closed) tier
        prev = 0
        for k in range(dbits + 1):
            t = orc.tier_of(k, dbits, T)
            assert 0 <= t <= T - 1 and t >= prev
            # equal-width intervals over [0, 1]: sim in [t/T, (t+1)/T)
            if k < dbits:
                assert t / T <= k / dbits < (t + 1) / T + 1e-15
            prev = t
    assert [orc.tier_of(k, 128, 8) for k in (15, 16, 31, 32, 127)] == [0, 1, 1, 2, 7]


def test_simtier_is_a_histogram():
    g = np.random.default_rng(4)
    m = g.integers(0, 129, 1000)
    h = orc.simtier(m, 128, 8)
    assert h.sum() == 1000 and (h >= 0).all()
    assert np.array_equal(h, np.bincount(np.minimum(m // 16, 7), minlength=8))
    assert np.allclose(orc.simtier(m, 128, 8, orc.NORM_MEAN), h / 1000)
    assert np.array_equal(orc.simtier(np.full(10, 128), 128, 8), [0, 0, 0, 0, 0, 0, 0, 10])   # identical signatures
    assert np.array_equal(orc.simtier(np.zeros(10, int), 128, 8), [10, 0, 0, 0, 0, 0, 0, 0])  # complements


def test_lsh_din_special_cases():
    g = np.random.default_rng(5)
    S = g.standard_normal((9, 6))
    assert np.allclose(orc.lsh_din(np.ones(9), S), S.sum(0), atol=1e-14)
    assert np.allclose(orc.lsh_din(np.ones(9), S, orc.NORM_MEAN), S.mean(0), atol=1e-14)
    assert np.allclose(orc.lsh_din([0.25], S[:1]), 0.25 * S[0], atol=1e-15)
    onehot = np.zeros(9); onehot[4] = 1.0
    assert np.array_equal(orc.lsh_din(onehot, S), S[4])
    sim = g.random(9)
    assert np.allclose(orc.lsh_din(sim, S), sim @ S, atol=1e-13)


# ------------------------------------------------------------------------------------------------
# attention (dense target attention; eqs. 2-3 share the routine)
# ------------------------------------------------------------------------------------------------
def test_attention_special_cases():
    g = np.random.default_rng(6)
    d = 8
    S = g.standard_normal((11, d))
    q = g.standard_normal(d)
    assert np.array_equal(orc.attention(q, S[:1]), S[0])                       # l = 1
    assert np.allclose(orc.attention(np.zeros(d), S), S.mean(0), atol=1e-15)   # zero query -> plain mean
    same = np.tile(S[3], (5, 1))
    assert np.allclose(orc.attention(q, same), S[3], atol=1e-15)               # identical rows
    att = orc.attention(q, S)
    assert (att <= S.max(0) + 1e-12).all() and (att >= S.min(0) - 1e-12).all() # convex combination
    delta = g.standard_normal(d)
    assert np.allclose(orc.attention(q, S + delta), att + delta, atol=1e-12)   # common score shift cancels
    big = orc.attention(1000.0 * q, S)                                         # no overflow; -> arg max row
    assert np.isfinite(big).all() and np.allclose(big, S[np.argmax(S @ q)], atol=1e-9)


def test_attention_closed_form_two_keys_fixes_the_scale():
    # d = 4, q = (2,0,0,0): score difference = 2 * (S0 - S1)[0] / sqrt(4) = ln 3  ->  weights 3/4, 1/4
    S = np.array([[math.log(3.0), 1.0, 0.0, 5.0], [0.0, -1.0, 2.0, 1.0]])
    q = np.array([2.0, 0.0, 0.0, 0.0])
    assert np.allclose(orc.attention(q, S), 0.75 * S[0] + 0.25 * S[1], atol=1e-14)
    # the query multiplies S_j (not the other way round): a query along axis 1 prefers row 0 (entry +1 vs -1)
    q2 = np.array([0.0, 2.0, 0.0, 0.0])
    w0 = 1.0 / (1.0 + math.exp(-2.0))
    assert np.allclose(orc.attention(q2, S), w0 * S[0] + (1 - w0) * S[1], atol=1e-14)


def test_attention_against_library_softmax():
    g = np.random.default_rng(7)
    S = g.standard_normal((50, 16)); q = g.standard_normal(16)
    s = S @ q / 4.0
    a = np.exp(s - s.max()); a /= a.sum()
    assert np.allclose(orc.attention(q, S), a @ S, atol=1e-13)


# ------------------------------------------------------------------------------------------------
# BEA (Algorithm 1, line 4)
# ------------------------------------------------------------------------------------------------
def test_bea_special_cases():
    g = np.random.default_rng(8)
    V = g.standard_normal((8, 5))
    for k in range(8):
        w = np.zeros(8); w[k] = 1.0
        assert np.array_equal(orc.bea(w, V), V[k])                    # one-hot weight picks a row of V
    w = g.dirichlet(np.ones(8))
    assert np.allclose(orc.bea(w, np.tile(V[2], (8, 1))), V[2], atol=1e-15)
    out = orc.bea(w, V)
    assert (out <= V.max(0) + 1e-12).all() and (out >= V.min(0) - 1e-12).all()
    assert np.allclose(orc.bea([2.0], V[:1]), 2.0 * V[0])             # n = 1
    assert np.allclose(orc.bea([0.5, 0.25], np.array([[1.0, 2.0], [4.0, 8.0]])), [1.5, 3.0])


# ------------------------------------------------------------------------------------------------
# bucket hash
# ------------------------------------------------------------------------------------------------
def test_mix64_against_published_splitmix64_vectors(golden_dir):
    GOLD = 0x9E3779B97F4A7C15
    for ln in open(os.path.join(golden_dir, "splitmix64_vectors.txt")):
        if ln[0] == "#":
            continue
        seed, k, out = ln.split()
        seed, k = int(seed), int(k)
        if seed == 0:
            assert orc.mix64(k, 0) == int(out, 16)                    # state = k * GOLD
        # state = seed + k * GOLD: reached as id = k, field = seed
        assert orc.mix64(k, seed) == int(out, 16)
    assert GOLD == 11400714819323198485


def test_bucket_modes():
    assert [orc.bucket(i, 3, 16, orc.BUCKET_MOD) for i in (0, 15, 16, 99999)] == [0, 15, 0, 99999 % 16]
    for i in (0, 1, 12345, 9_999_999):
        for f in (0, 1, 63):
            assert orc.bucket(i, f, 4096, orc.BUCKET_HASH) == orc.mix64(i, f) % 4096
    # fields decorrelate: the buckets of one id over 64 fields are not all equal
    assert len({orc.bucket(777, f, 4096, orc.BUCKET_HASH) for f in range(64)}) > 32


# ------------------------------------------------------------------------------------------------
# MLP
# ------------------------------------------------------------------------------------------------
def _tiny_cfg(**kw):
    base = dict(dtype=orc.F32, M=10, d=2, F=0, B=1, dc=0, hidden=(3, 2), blocks=0)
    base.update(kw)
    return orc.OracleConfig(**base)


def _mlp(cfg, W, b, w_out, b_out):
    return orc.Oracle(cfg, {"W": [np.asarray(w, np.float32) for w in W], "b": [np.asarray(x, np.float32) for x in b],
                            "w_out": np.asarray(w_out, np.float32), "b_out": np.asarray([b_out], np.float32)})


def test_mlp_hand_worked():
    cfg = _tiny_cfg()
    assert cfg.input_width() == 4
    W1 = [[1, 0, 0, 0], [0, -1, 0, 2], [1, 1, 1, 1]]
    W2 = [[1, 1, 0], [0, -1, 0.5]]
    o = _mlp(cfg, [W1, W2], [[0, 0.5, -10], [0.25, 0]], [2, -4], 0.125)
    x = [1.0, 2.0, 3.0, 0.5]
    # h1 = relu([1, -2+1+0.5, 6.5-10]) = [1, 0, 0]; h2 = relu([1+0.25, 0]) = [1.25, 0]; logit = 2.5 + 0.125
    assert o.mlp(x) == 2.625
    x = [-1.0, -2.0, 30.0, 0.0]
    # h1 = relu([-1, 2.5, 17]) = [0, 2.5, 17]; h2 = relu([2.75, 6]) ; logit = 5.5 - 24 + .125
    assert o.mlp(x) == 5.5 - 24 + 0.125


def test_mlp_zero_weights_and_sigmoid():
    cfg = _tiny_cfg()
    z = _mlp(cfg, [np.zeros((3, 4)), np.zeros((2, 3))], [np.zeros(3), np.zeros(2)], [0, 0], 0.75)
    assert z.mlp([5, 6, 7, 8]) == 0.75
    s = _mlp(_tiny_cfg(emit_sigmoid=1), [np.zeros((3, 4)), np.zeros((2, 3))], [np.zeros(3), np.zeros(2)], [0, 0], 0.0)
    assert s.mlp([1, 2, 3, 4]) == 0.5
    s2 = _mlp(_tiny_cfg(emit_sigmoid=1), [np.zeros((3, 4)), np.zeros((2, 3))], [np.zeros(3), np.zeros(2)], [0, 0],
              math.log(3.0))
    assert abs(s2.mlp([0, 0, 0, 0]) - 0.75) < 1e-7     # b_out is stored as fp32


def test_mlp_three_hidden_layers():
    cfg = _tiny_cfg(hidden=(2, 2, 2))
    o = _mlp(cfg, [[[1, 0, 0, 0], [0, 1, 0, 0]], [[0, 1], [1, 0]], [[1, 1], [1, -1]]], [[0, 0]] * 3, [1, 10], 0)
    # x = [3, 5, ., .] -> h1 = [3, 5] -> h2 = [5, 3] -> h3 = [8, 2] -> 8 + 20
    assert o.mlp([3, 5, 9, 9]) == 28.0


# ------------------------------------------------------------------------------------------------
# concatenation order and every block's placement, through selector weights
# ------------------------------------------------------------------------------------------------
def _selector_oracle(wl, col, sign=1.0):
    width = wl.input_width()
    W1 = np.zeros((wl.hidden[0], width), np.float32); W1[0, col] = sign
    W2 = np.zeros((wl.hidden[1], wl.hidden[0]), np.float32); W2[0, 0] = 1.0
    w_out = np.zeros(wl.hidden[1], np.float32); w_out[0] = 1.0
    mlp = {"W": [W1, W2], "b": [np.zeros(wl.hidden[0], np.float32), np.zeros(wl.hidden[1], np.float32)],
           "w_out": w_out, "b_out": np.zeros(1, np.float32)}
    return orc.Oracle(helpers.oracle_config(wl), mlp)


def test_concat_layout_by_selector_weights():
    wl = synth.Workload("sel", "f32", R=1, N=4, M=50, d=8, L=1, F=3, B=5, dc=2, hidden=(2, 2), sigma=1.0,
                        bucket_mode=synth.BUCKET_MOD, id_dist="uniform", blocks=helpers.ALL_BLOCKS, n_bridge=3,
                        n_tiers=4, lsh_din_norm=synth.NORM_NONE, simtier_norm=synth.NORM_NONE)
    tab = synth.make_item_table(wl)
    rq = synth.make_request(wl, 0)
    # one-hot BEA weights, sequence of length 1, identical signatures: every block has a hand-known value
    cid = 13
    bea_w = np.zeros((wl.M, 3), np.float32); bea_w[:, 1] = 1.0
    tab["bea_w"] = bea_w
    tab["sig"][:] = 0xA5
    rq["sig_seq"][:] = 0xA5
    E, u, S, T, V = tab["E"], rq["u"], rq["S"], rq["T"], rq["V"]
    expect = np.concatenate([
        u, E[cid], S[0],                                   # user | item | attention over one key = that key
        T[0, cid % 5], T[1, cid % 5], T[2, cid % 5],       # cross fields in order
        V[1],                                              # BEA: one-hot weight picks V[1]
        1.0 * S[0],                                        # LSH-DIN: sim = 1, l = 1
        [0, 0, 0, 1],                                      # SimTier: the one similarity (=1) falls in the last tier
    ]).astype(np.float64)
    assert expect.size == wl.input_width() == 8 + 8 + 8 + 6 + 8 + 8 + 4
    req = helpers.projected_request(wl, rq)
    for col in range(expect.size):
        for sign in (1.0, -1.0):
            got = _selector_oracle(wl, col, sign).score(tab, req, [cid])[0]
            assert got == max(0.0, sign * expect[col]), (col, sign)
    _, x = _selector_oracle(wl, 0).score(tab, req, [cid], return_inputs=True)
    assert np.array_equal(x[0], expect)


# ------------------------------------------------------------------------------------------------
# invariants of the method
# ------------------------------------------------------------------------------------------------
@pytest.fixture(scope="module")
def small():
    wl = synth.Workload("inv", "bf16", R=2, N=64, M=500, d=16, L=12, F=4, B=32, dc=8, hidden=(32, 16), sigma=0.3,
                        blocks=helpers.ALL_BLOCKS, dU=24)
    w = synth.make_weights(wl, zero_bias=False)
    tab = synth.make_item_table(wl)
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    o = helpers.make_oracle(wl, w)
    return wl, w, tab, rq, ids, o


def test_decomposed_first_layer_equals_concatenated(small):
    wl, w, tab, rq, ids, o = small
    req = helpers.raw_request(o, rq)
    logits, x = o.score(tab, req, ids, return_inputs=True)
    W1 = synth.as_f32(w["mlp"]["W"][0], wl.dtype).astype(np.float64)
    W2 = synth.as_f32(w["mlp"]["W"][1], wl.dtype).astype(np.float64)
    wo = synth.as_f32(w["mlp"]["w_out"], wl.dtype).astype(np.float64)
    b1, b2 = w["mlp"]["b"][0].astype(np.float64), w["mlp"]["b"][1].astype(np.float64)
    d = wl.d
    p_u = W1[:, :d] @ req["u"] + b1                       # user partial product, once per request
    pre = p_u[None, :] + x[:, d:] @ W1[:, d:].T           # + candidate-dependent part
    full = x @ W1.T + b1
    assert np.allclose(pre, full, rtol=1e-12, atol=1e-14)
    h2 = np.maximum(np.maximum(pre, 0) @ W2.T + b2, 0)
    assert np.allclose(h2 @ wo + float(w["mlp"]["b_out"][0]), logits, rtol=1e-12, atol=1e-14)


def test_permutation_equivariance_and_minibatch_split(small):
    wl, w, tab, rq, ids, o = small
    req = helpers.raw_request(o, rq)
    whole = o.score(tab, req, ids)
    perm = np.random.default_rng(9).permutation(ids.size)
    assert np.array_equal(o.score(tab, req, ids[perm]), whole[perm])
    parts = np.concatenate([o.score(tab, req, ids[s:s + 10]) for s in range(0, ids.size, 10)])
    assert np.array_equal(parts, whole)


def test_cached_user_state_equals_recomputed(small):
    wl, w, tab, rq, ids, o = small
    u1, S1 = o.user_state(rq["profile"], rq["seq"])
    u2, S2 = o.user_state(rq["profile"], rq["seq"])
    assert np.array_equal(u1, u2) and np.array_equal(S1, S2)
    a = o.score(tab, {**helpers.raw_request(o, rq)}, ids)
    b = o.score(tab, {"u": u1, "S": S1, "T": rq["T"], "V": rq["V"], "sig_seq": rq["sig_seq"]}, ids)
    assert np.array_equal(a, b)


def test_out_of_range_ids_give_nan(small):
    wl, w, tab, rq, ids, o = small
    req = helpers.raw_request(o, rq)
    bad = np.array([ids[0], -1, wl.M, ids[1]], np.int32)
    out = o.score(tab, req, bad)
    assert o.last_bad == 2 and np.isnan(out[1]) and np.isnan(out[2])
    assert np.array_equal(out[[0, 3]], o.score(tab, req, ids[:2]))


# ------------------------------------------------------------------------------------------------
# user-side network, eqs. 1-3
# ------------------------------------------------------------------------------------------------
def _user_oracle(d, dU, Wp, Ws, Wa, ba, Wb, bb):
    cfg = orc.OracleConfig(dtype=orc.F32, M=1, d=d, hidden=(1,), blocks=0)
    mlp = {"W": [np.zeros((1, 2 * d), np.float32)], "b": [np.zeros(1, np.float32)],
           "w_out": np.zeros(1, np.float32), "b_out": np.zeros(1, np.float32)}
    f = lambda a: np.asarray(a, np.float32)
    return orc.Oracle(cfg, mlp, {"W_profile": f(Wp), "W_seq": f(Ws), "W_a": f(Wa), "b_a": f(ba), "W_b": f(Wb),
                                 "b_b": f(bb)})


def test_user_state_special_cases():
    g = np.random.default_rng(10)
    d = dU = 4
    I = np.eye(d)
    seq = g.standard_normal((6, dU)).astype(np.float32)
    prof = g.standard_normal(dU).astype(np.float32)
    # identity projections, FFN that outputs only its bias: u = b_b + profile attention
    bb = np.array([1, 2, 3, 4.0])
    o = _user_oracle(d, dU, I, I, I, np.zeros(d), np.zeros((d, d)), bb)
    u, S = o.user_state(prof, seq)
    assert np.array_equal(S, seq.astype(np.float64))
    assert np.allclose(u, bb + orc.attention(prof.astype(np.float64), S), atol=1e-14)
    # l = 1: both attentions return the single projected row s; u = FFN(s) + s
    Ws = g.standard_normal((d, dU)).astype(np.float32)
    Wa = g.standard_normal((d, d)).astype(np.float32)
    Wb = g.standard_normal((d, d)).astype(np.float32)
    ba = g.standard_normal(d).astype(np.float32)
    o = _user_oracle(d, dU, g.standard_normal((d, dU)), Ws, Wa, ba, Wb, bb)
    u, S = o.user_state(prof, seq[:1])
    s = seq[0].astype(np.float64) @ Ws.astype(np.float64).T       # U_seq W_seq^T: weight rows index the output
    assert np.allclose(S[0], s, atol=1e-14)
    ffn = np.maximum(s @ Wa.astype(np.float64).T + ba, 0) @ Wb.astype(np.float64).T + bb
    assert np.allclose(u, ffn + s, atol=1e-13)


def test_user_state_against_library_ops():
    g = np.random.default_rng(11)
    d, dU, l = 8, 5, 17
    Wp, Ws = g.standard_normal((d, dU)).astype(np.float32), g.standard_normal((d, dU)).astype(np.float32)
    Wa, Wb = g.standard_normal((d, d)).astype(np.float32), g.standard_normal((d, d)).astype(np.float32)
    ba, bb = g.standard_normal(d).astype(np.float32), g.standard_normal(d).astype(np.float32)
    seq, prof = g.standard_normal((l, dU)).astype(np.float32), g.standard_normal(dU).astype(np.float32)
    u, S = _user_oracle(d, dU, Wp, Ws, Wa, ba, Wb, bb).user_state(prof, seq)
    f = lambda a: a.astype(np.float64)

    def softmax(z):
        e = np.exp(z - z.max(-1, keepdims=True))
        return e / e.sum(-1, keepdims=True)
    Sh, ph = f(seq) @ f(Ws).T, f(prof) @ f(Wp).T
    ctx = softmax(Sh @ Sh.T / math.sqrt(d)) @ Sh
    Z = np.maximum(ctx @ f(Wa).T + f(ba), 0) @ f(Wb).T + f(bb)
    expect = Z.mean(0) + softmax(ph @ Sh.T / math.sqrt(d)) @ Sh
    assert np.allclose(S, Sh, atol=1e-13) and np.allclose(u, expect, atol=1e-12)


# ------------------------------------------------------------------------------------------------
# brute force on a tiny input, in plain Python
# ------------------------------------------------------------------------------------------------
def test_whole_path_brute_force_tiny():
    wl = synth.Workload("brute", "f32", R=1, N=5, M=40, d=3, L=4, F=2, B=7, dc=2, hidden=(4, 3), sigma=0.8,
                        bucket_mode=synth.BUCKET_HASH, id_dist="uniform", blocks=helpers.ALL_BLOCKS, n_bridge=2,
                        n_tiers=3, lsh_din_norm=synth.NORM_MEAN, simtier_norm=synth.NORM_NONE)
    wl = wl.with_(d=8)          # signatures need a whole number of bytes: d' = d = 8
    w = synth.make_weights(wl, zero_bias=False)
    tab, rq = synth.make_item_table(wl), synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    o = helpers.make_oracle(wl, w)
    got = o.score(tab, helpers.projected_request(wl, rq), ids)

    d, L = wl.d, wl.L
    fl = lambda a: [[float(v) for v in row] for row in np.atleast_2d(a)]
    E, S, V, bw = fl(tab["E"]), fl(rq["S"]), fl(rq["V"]), fl(tab["bea_w"])
    u = [float(v) for v in rq["u"]]
    W = [fl(m) for m in w["mlp"]["W"]]
    b = [[float(v) for v in m] for m in w["mlp"]["b"]]
    wo, bo = [float(v) for v in w["mlp"]["w_out"]], float(w["mlp"]["b_out"][0])
    MASK = 2**64 - 1

    def h64(i, f):
        z = (i * 0x9E3779B97F4A7C15 + f) & MASK
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
        return z ^ (z >> 31)

    for n, c in enumerate(int(i) for i in ids):
        e = E[c]
        s = [sum(e[k] * S[j][k] for k in range(d)) / math.sqrt(d) for j in range(L)]
        z = sum(math.exp(v) for v in s)
        att = [sum(math.exp(s[j]) / z * S[j][k] for j in range(L)) for k in range(d)]
        cross = []
        for f in range(wl.F):
            cross += [float(v) for v in rq["T"][f, h64(c, f) % wl.B]]
        vb = [sum(bw[c][k] * V[k][j] for k in range(wl.n_bridge)) for j in range(d)]
        bits_c = format(int(tab["sig"][c, 0]), "08b")
        match = [sum(1 for p in range(8) if bits_c[p] == format(int(rq["sig_seq"][j, 0]), "08b")[p]) for j in range(L)]
        din = [sum(match[j] / 8.0 * S[j][k] for j in range(L)) / L for k in range(d)]
        tiers = [0.0] * 3
        for m in match:
            tiers[min(2, (m * 3) // 8)] += 1.0
        x = u + e + att + cross + vb + din + tiers
        a = x
        for k in range(2):
            a = [max(0.0, sum(W[k][r][i] * a[i] for i in range(len(a))) + b[k][r]) for r in range(len(W[k]))]
        logit = sum(wo[i] * a[i] for i in range(len(a))) + bo
        assert abs(got[n] - logit) < 1e-12


# ------------------------------------------------------------------------------------------------
# item table write (nearline refresh)
# ------------------------------------------------------------------------------------------------
def test_table_refresh_full_and_incremental():
    g = np.random.default_rng(12)
    table = np.zeros((20, 8), np.uint16)
    rows = g.integers(0, 65535, (20, 8)).astype(np.uint16)
    assert orc.table_refresh(table, None, rows) == 0 and np.array_equal(table, rows)
    upd = g.integers(0, 65535, (4, 8)).astype(np.uint16)
    ids = np.array([3, 25, -2, 7], np.int32)
    assert orc.table_refresh(table, ids, upd) == 2
    expect = rows.copy(); expect[3] = upd[0]; expect[7] = upd[3]
    assert np.array_equal(table, expect)


def test_bf16_storage_is_widened_exactly():
    a = np.array([1.0, -0.3330078125, 3.0e-5, 65280.0], np.float32)
    bits = synth.to_bf16_bits(a)
    assert np.array_equal(orc.widen(bits, orc.BF16), synth.bf16_bits_to_f32(bits).astype(np.float64))
    # round to nearest even on the 16 dropped bits
    assert synth.to_bf16_bits(np.array([1.00390625], np.float32))[0] == 0x3F80      # tie -> even (down)
    assert synth.to_bf16_bits(np.array([1.01171875], np.float32))[0] == 0x3F82      # tie -> even (up)


# ------------------------------------------------------------------------------------------------
# item side of the nearline pipeline (Section 3.2 eq. 4, Algorithm 1 step 3, Section 4.2 eq. 5)
# ------------------------------------------------------------------------------------------------
def test_item_tower_special_cases_and_brute_force():
    g = np.random.default_rng(11)
    n, dI, hI, d = 5, 12, 7, 4
    I = g.standard_normal((n, dI)).astype(np.float32)
    W0 = g.standard_normal((hI, dI)).astype(np.float32)
    b0 = g.standard_normal(hI).astype(np.float32)
    W1 = g.standard_normal((d, hI)).astype(np.float32)
    b1 = g.standard_normal(d).astype(np.float32)
    got = orc.item_nearline(orc.F32, I_raw=I, W0=W0, b0=b0, W1=W1, b1=b1)["I_hat"]
    # brute force, scalar loops
    for i in range(n):
        h = [max(0.0, float(b0[j]) + sum(float(W0[j, c]) * float(I[i, c]) for c in range(dI))) for j in range(hI)]
        for k in range(d):
            want = float(b1[k]) + sum(float(W1[k, j]) * h[j] for j in range(hI))
            assert abs(got[i, k] - want) < 1e-12
    # zero first layer: the output is W1 ReLU(b0) + b1 for every item
    z = orc.item_nearline(orc.F32, I_raw=I, W0=np.zeros_like(W0), b0=b0, W1=W1, b1=b1)["I_hat"]
    assert np.allclose(z, (W1.astype(np.float64) @ np.maximum(b0.astype(np.float64), 0) + b1)[None, :], atol=1e-12)
    # all pre-activations positive: the network is affine, I^ = W1 (W0 I + b0) + b1
    big = np.full(hI, 100.0, dtype=np.float32)
    a = orc.item_nearline(orc.F32, I_raw=I, W0=W0, b0=big, W1=W1, b1=b1)["I_hat"]
    want = (W1.astype(np.float64) @ (W0.astype(np.float64) @ I.astype(np.float64).T + big[:, None].astype(np.float64))).T + b1
    assert np.allclose(a, want, atol=1e-10)
    # all pre-activations negative: only the output bias is left
    neg = orc.item_nearline(orc.F32, I_raw=I, W0=W0, b0=-big, W1=W1, b1=b1)["I_hat"]
    assert np.allclose(neg, b1[None, :].astype(np.float64), atol=0)
    # a hidden unit that is negative for one sign of the input and positive for the other: ReLU sits between the layers
    one = orc.item_nearline(orc.F32, I_raw=np.array([[1.0], [-1.0]], np.float32), W0=np.array([[2.0]], np.float32),
                            b0=np.zeros(1, np.float32), W1=np.array([[3.0]], np.float32), b1=np.zeros(1, np.float32))["I_hat"]
    assert one[0, 0] == 6.0 and one[1, 0] == 0.0


def test_item_bridge_weights_are_a_softmax_over_the_bridges():
    g = np.random.default_rng(12)
    n, d, nb = 6, 16, 8
    I = g.standard_normal((n, d)).astype(np.float32)
    Bm = g.standard_normal((nb, d)).astype(np.float32)
    w = orc.item_nearline(orc.F32, I_id=I, bridges=Bm)["w_hat"]
    assert w.shape == (n, nb) and np.allclose(w.sum(axis=1), 1.0, atol=1e-14) and (w > 0).all()
    # closed form against a hand-written softmax of I B^T / sqrt(d) (item rows times bridge rows: not B I^T transposed wrongly)
    s = (I.astype(np.float64) @ Bm.astype(np.float64).T) / math.sqrt(d)
    e = np.exp(s - s.max(axis=1, keepdims=True))
    assert np.allclose(w, e / e.sum(axis=1, keepdims=True), atol=1e-14)
    # equal bridges: uniform weights; a bridge equal to a large multiple of the item: weight near one
    u = orc.item_nearline(orc.F32, I_id=I, bridges=np.tile(Bm[:1], (nb, 1)))["w_hat"]
    assert np.allclose(u, 1.0 / nb, atol=1e-15)
    Bs = np.zeros((nb, d), np.float32)
    Bs[3] = 50.0 * I[2]
    assert orc.item_nearline(orc.F32, I_id=I, bridges=Bs)["w_hat"][2, 3] > 0.999
    # the scale is 1 / sqrt(d): with d = 4 and products (2 ln 3, 0) the scores are (ln 3, 0), the weights (3, 1) / 4
    I2 = np.array([[1.0, 0.0, 0.0, 0.0]], np.float32)
    B2 = np.array([[2.0 * math.log(3.0), 0, 0, 0], [0, 0, 0, 0]], np.float32)
    w2 = orc.item_nearline(orc.F32, I_id=I2, bridges=B2)["w_hat"]
    assert np.allclose(w2, [[0.75, 0.25]], atol=1e-6)
    # Algorithm 1 step 4 on top: with one-hot weights the weighted sum picks a user-side vector
    V = g.standard_normal((nb, d))
    onehot = np.zeros(nb); onehot[5] = 1.0
    assert np.array_equal(orc.bea(onehot, V), V[5])


def test_item_signatures_pack_eq5_bits_first_bit_most_significant():
    g = np.random.default_rng(13)
    n, d_mm, dbits = 9, 24, 64
    M = g.standard_normal((n, d_mm)).astype(np.float32)
    W = g.standard_normal((dbits, d_mm)).astype(np.float32)
    sig = orc.item_nearline(orc.F32, M_mm=M, W_hash=W)["sig"]
    proj = orc.lsh_projections(orc.F32, M, W)
    assert np.allclose(proj, M.astype(np.float64) @ W.astype(np.float64).T, atol=1e-12)
    for i in range(n):
        bits = orc.lsh_hash_bits(M[i], W)
        assert np.array_equal(bits, (proj[i] > 0).astype(np.uint8))
        assert np.array_equal(sig[i], np.packbits(bits))        # numpy packs big-endian: first bit = most significant
        assert np.array_equal(sig[i], orc.pack_bits(bits))
    # an item whose first eight projections have the signs 0 0 1 1 0 1 0 1 gets the byte 53 (Section 4.2's example)
    Wd = np.zeros((8, 8), np.float32)
    for k, b in enumerate([0, 0, 1, 1, 0, 1, 0, 1]):
        Wd[k, k] = 1.0 if b else -1.0
    s53 = orc.item_nearline(orc.F32, M_mm=np.ones((1, 8), np.float32), W_hash=Wd)["sig"]
    assert s53.tolist() == [[53]]
    # similarity of an item with itself is 1, with its negation 0 (eq. 6 on the produced signatures)
    both = orc.item_nearline(orc.F32, M_mm=np.vstack([M[:1], -M[:1]]), W_hash=W)["sig"]
    sim = orc.lsh_similarity(both[:1], both, dbits)
    assert sim[0, 0] == 1.0 and sim[0, 1] == 0.0


def test_bea_user_side_and_the_whole_of_algorithm_1():
    g = np.random.default_rng(14)
    n, m, d, b = 4, 6, 8, 5
    Bm = g.standard_normal((n, d)).astype(np.float32)
    U = g.standard_normal((m, d)).astype(np.float32)
    Wf = g.standard_normal((d, d)).astype(np.float32)
    V, W = orc.bea_user(orc.F32, Bm, U, Wf)
    # step 1: one softmax per bridge over the user-side features (rows of B against rows of U)
    assert W.shape == (n, m) and np.allclose(W.sum(axis=1), 1.0, atol=1e-14) and (W > 0).all()
    s = Bm.astype(np.float64) @ U.astype(np.float64).T / math.sqrt(d)
    e = np.exp(s - s.max(axis=1, keepdims=True))
    assert np.allclose(W, e / e.sum(axis=1, keepdims=True), atol=1e-14)
    # step 2 under the reading V_k = W_f (sum_j W_kj U_j): brute force with scalar loops
    for k in range(n):
        a = [sum(W[k, j] * float(U[j, c]) for j in range(m)) for c in range(d)]
        for r in range(d):
            assert abs(V[k, r] - sum(float(Wf[r, c]) * a[c] for c in range(d))) < 1e-12
    # one user-side feature: every bridge sees weight 1, V_k = W_f U_0 for every k
    V1, W1 = orc.bea_user(orc.F32, Bm, U[:1], Wf)
    assert np.array_equal(W1, np.ones((n, 1)))
    assert np.allclose(V1, np.tile(Wf.astype(np.float64) @ U[0].astype(np.float64), (n, 1)), atol=1e-13)
    # identity W_f: V_k is a convex combination of the rows of U; a bridge far along one feature picks that feature
    Vi, _ = orc.bea_user(orc.F32, Bm, U, np.eye(d, dtype=np.float32))
    assert (Vi <= U.max(axis=0) + 1e-12).all() and (Vi >= U.min(axis=0) - 1e-12).all()
    Bs = Bm.copy(); Bs[2] = 60.0 * U[4]
    Vs, Ws = orc.bea_user(orc.F32, Bs, U, np.eye(d, dtype=np.float32))
    assert Ws[2, 4] > 0.999 and np.allclose(Vs[2], U[4], atol=1e-2)
    # the whole algorithm: v^ = Softmax(I B^T / sqrt d) V, composed from the item-side and user-side oracles
    I = g.standard_normal((b, d)).astype(np.float32)
    w_hat = orc.item_nearline(orc.F32, I_id=I, bridges=Bm)["w_hat"]
    for i in range(b):
        assert np.allclose(orc.bea(w_hat[i], V), w_hat[i] @ V, atol=1e-13)
    # with a single bridge the approximation collapses to the same vector for every item
    V0, _ = orc.bea_user(orc.F32, Bm[:1], U, Wf)
    w0 = orc.item_nearline(orc.F32, I_id=I, bridges=Bm[:1])["w_hat"]
    assert np.array_equal(w0, np.ones((b, 1))) and np.allclose(orc.bea(w0[3], V0), V0[0], atol=0)


# ------------------------------------------------------------------------------------------------
# Category sub-sequences (Section 3.3, SIM-hard): the interaction blocks restricted to the behaviours whose category is
# the candidate's
# ------------------------------------------------------------------------------------------------
def _sim_setup(n_categories, L=40, N=60, blocks=helpers.ALL_BLOCKS, seed=0, dtype="f32"):
    base = synth.C1 if dtype == "f32" else synth.C2
    wl = base.with_(name=f"sim_pin_{n_categories}_{seed}", N=N, M=500, L=L, blocks=blocks, n_categories=n_categories,
                    lsh_din_norm=synth.NORM_MEAN, simtier_norm=synth.NORM_MEAN, emit_sigmoid=0, hidden=(32, 16), F=2, B=8, dc=8)
    weights = synth.make_weights(wl, zero_bias=False)
    table = synth.make_item_table(wl)
    rq = synth.make_request(wl, seed)
    ids = synth.IdSampler(wl).request_ids(seed)
    return wl, weights, table, rq, ids


def test_category_is_the_bucket_function_on_its_own_field():
    for i in (0, 1, 17, 4242, 2**31 - 1):
        for C_ in (1, 7, 100):
            assert orc.category(i, C_, orc.BUCKET_MOD) == i % C_
            assert orc.category(i, C_, orc.BUCKET_HASH) == orc.mix64(i, orc.CATEGORY_FIELD) % C_
            assert orc.category(i, C_, orc.BUCKET_HASH) == orc.bucket(i, orc.CATEGORY_FIELD, C_, orc.BUCKET_HASH)


def test_one_category_is_the_whole_sequence():
    wl, weights, table, rq, ids = _sim_setup(1)
    assert (rq["seq_cat"] == 0).all()
    with_cat = helpers.make_oracle(wl, weights).score(table, helpers.projected_request(wl, rq), ids)
    plain_wl = wl.with_(n_categories=0)
    plain = helpers.make_oracle(plain_wl, weights).score(table, helpers.projected_request(plain_wl, rq), ids)
    assert np.array_equal(with_cat, plain)


def test_every_behaviour_in_the_candidates_category_is_the_whole_sequence_and_none_is_all_zeros():
    wl, weights, table, rq, ids = _sim_setup(5)
    oracle = helpers.make_oracle(wl, weights)
    plain_wl = wl.with_(n_categories=0)
    plain, xp = helpers.make_oracle(plain_wl, weights).score(table, helpers.projected_request(plain_wl, rq), ids, return_inputs=True)
    d = wl.d
    for i in (0, 7, 31):
        cat = orc.category(int(ids[i]), 5, wl.bucket_mode)
        rq_all = dict(rq, seq_cat=np.full(wl.L, cat, dtype=np.int32))
        got, x = oracle.score(table, helpers.projected_request(wl, rq_all), ids[i:i + 1], return_inputs=True)
        assert got[0] == plain[i] and np.array_equal(x[0], xp[i])
        rq_none = dict(rq, seq_cat=np.full(wl.L, (cat + 1) % 5, dtype=np.int32))
        _, x0 = oracle.score(table, helpers.projected_request(wl, rq_none), ids[i:i + 1], return_inputs=True)
        assert np.all(x0[0, 2 * d:3 * d] == 0.0)                       # attention
        tail = x0[0, 3 * d + wl.F * wl.dc + d:]                        # [lsh_din | simtier] after cross and v_bea
        assert tail.shape[0] == d + wl.n_tiers and np.all(tail == 0.0)
        assert np.array_equal(x0[0, :2 * d], xp[i, :2 * d])            # u and e do not depend on the sequence


def test_a_sub_sequence_of_one_item_gives_that_item():
    wl, weights, table, rq, ids = _sim_setup(3)
    oracle = helpers.make_oracle(wl, weights)
    i = 4
    cat = orc.category(int(ids[i]), 3, wl.bucket_mode)
    seq_cat = np.full(wl.L, (cat + 1) % 3, dtype=np.int32)
    seq_cat[11] = cat
    _, x = oracle.score(table, helpers.projected_request(wl, dict(rq, seq_cat=seq_cat)), ids[i:i + 1], return_inputs=True)
    d = wl.d
    S = synth.as_f32(rq["S"], wl.dtype).astype(np.float64)
    assert np.allclose(x[0, 2 * d:3 * d], S[11], rtol=0, atol=1e-15)   # softmax over one key is 1
    k = orc.lsh_matches(table["sig"][ids[i]], rq["sig_seq"][11])
    off = 3 * d + wl.F * wl.dc + d
    assert np.allclose(x[0, off:off + d], (k / wl.lsh_bits) * S[11], rtol=0, atol=1e-15)   # mean over one item
    tiers = x[0, off + d:]
    assert tiers.sum() == 1.0 and tiers[orc.tier_of(k, wl.lsh_bits, wl.n_tiers)] == 1.0


def test_sub_sequences_against_explicit_selection_and_under_a_permutation_of_the_sequence():
    wl, weights, table, rq, ids = _sim_setup(4, L=57, seed=2)
    oracle = helpers.make_oracle(wl, weights)
    req = helpers.projected_request(wl, rq)
    want, x = oracle.score(table, req, ids, return_inputs=True)
    S = req["S"]
    d = wl.d
    E = synth.as_f32(table["E"], wl.dtype).astype(np.float64)
    for i in range(0, len(ids), 9):
        cat = int(ids[i]) % 4 if wl.bucket_mode == synth.BUCKET_MOD else orc.mix64(int(ids[i]), orc.CATEGORY_FIELD) % 4
        sel = np.flatnonzero(rq["seq_cat"] == cat)
        if len(sel) == 0:
            assert np.all(x[i, 2 * d:3 * d] == 0.0)
            continue
        # plain numpy: softmax(e S_c^T / sqrt(d)) S_c over the selected rows
        s = S[sel] @ E[ids[i]] / math.sqrt(d)
        a = np.exp(s - s.max())
        a /= a.sum()
        assert np.allclose(x[i, 2 * d:3 * d], a @ S[sel], rtol=0, atol=1e-14)
        k = np.array([orc.lsh_matches(table["sig"][ids[i]], rq["sig_seq"][j]) for j in sel])
        off = 3 * d + wl.F * wl.dc + d
        assert np.allclose(x[i, off:off + d], (k / wl.lsh_bits) @ S[sel] / len(sel), rtol=0, atol=1e-14)
        hist = np.bincount([orc.tier_of(int(v), wl.lsh_bits, wl.n_tiers) for v in k], minlength=wl.n_tiers) / len(sel)
        assert np.allclose(x[i, off + d:], hist, rtol=0, atol=1e-15)
    # the order of the behaviours does not matter, as long as every row keeps its category and its signature
    perm = np.random.default_rng(4).permutation(wl.L)
    rq_p = dict(rq, S=rq["S"][perm], sig_seq=rq["sig_seq"][perm], seq_cat=rq["seq_cat"][perm])
    got = oracle.score(table, helpers.projected_request(wl, rq_p), ids)
    assert np.abs(got - want).max() < 1e-12
