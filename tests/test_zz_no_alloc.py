"""aif_score_noalloc: the scoring entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits after start-up (a plug-in in a serving process whose
pool owns the whole GPU; a request thread that must stay out of the driver's allocator).  For them the library
offers a scoring call whose intermediate activations live in a fixed device array inside the library image.  This
test drives that call through the C ABI, twice in a row on the shared array, and checks each result against the
ordinary aif_score on the same inputs and against the CPU oracle; a third call, on a context whose own scratch is
much smaller, uses the fixed array up to its last row.  It is collected last on purpose, and it builds everything it
needs itself, so it passes alone in a fresh process as well as after the rest of the suite."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2511_12934_b200 import binding as B
from paper_2511_12934_b200 import build as libbuild
from paper_2511_12934_b200 import serving, synth
from tests import helpers

pytestmark = pytest.mark.gpu

TOL = 2e-3   # the bf16 tolerance of the parity tests


def test_noalloc_scoring_matches_aif_score_on_two_calls_in_a_row():
    libbuild.build()
    assert torch.cuda.is_available()
    wl = helpers.MINI["c2"].with_(name="noalloc", N=1000, blocks=helpers.ALL_BLOCKS)
    weights, table = synth.make_weights(wl), synth.make_item_table(wl)
    # aif_score (the reference here) uses the context's own scratch, so size that for the largest call
    srv = serving.Server(wl, weights, table, path=B.PATH_TENSOR, max_batch_candidates=1024)
    lib = srv.ctx.lib
    sampler = synth.IdSampler(wl)
    rq = synth.make_request(wl, 0)
    st = srv.precompute(7, srv.upload_request(rq, B.USER_PROJECTED))
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    oreq = helpers.projected_request(wl, rq)
    for call, n in enumerate((1000, 333)):                      # second call reuses the array the first one left dirty
        ids = torch.from_numpy(sampler.request_ids(call, n)).cuda()
        ref = torch.empty(n, dtype=torch.float32, device="cuda")
        out = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
        stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
        rc = lib.aif_score(srv.ctx.h, st.handle, C.c_void_p(ids.data_ptr()), n, C.c_void_p(ref.data_ptr()), stream)
        assert rc == B.OK
        rc = lib.aif_score_noalloc(srv.ctx.h, st.handle, C.c_void_p(ids.data_ptr()), n, C.c_void_p(out.data_ptr()), stream)
        assert rc == B.OK, lib.aif_last_error().decode()
        torch.cuda.synchronize()
        a, b = out.cpu().numpy(), ref.cpu().numpy()
        assert np.isfinite(a).all()
        assert np.abs(a - b).max() <= TOL, np.abs(a - b).max()
        want = oracle.score(table, oreq, ids.cpu().numpy())      # mini-batches of 500: ragged tiles inside the call
        assert np.abs(a - want).max() <= TOL, np.abs(a - want).max()
    assert srv.ctx.poll_status() == 0
    # sizes beyond the fixed array are refused with a clear message, nothing is launched
    big = torch.zeros(B.NOALLOC_MAX_CANDIDATES + 1, dtype=torch.int32, device="cuda")
    outb = torch.empty(big.numel(), dtype=torch.float32, device="cuda")
    before = B.kernel_launches()
    rc = lib.aif_score_noalloc(srv.ctx.h, st.handle, C.c_void_p(big.data_ptr()), big.numel(), C.c_void_p(outb.data_ptr()),
                               C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == B.ERR_SHAPE and "AIF_NOALLOC_MAX_CANDIDATES" in lib.aif_last_error().decode()
    assert B.kernel_launches() == before
    srv.close()
    # the call does not depend on the context's own scratch: a context sized for 256 candidates scores the fixed
    # array's maximum, which reaches its last row; the oracle is the checker (aif_score refuses this size here)
    small = serving.Server(wl, weights, table, path=B.PATH_TENSOR, max_batch_candidates=256)
    st2 = small.precompute(8, small.upload_request(rq, B.USER_PROJECTED))
    n = B.NOALLOC_MAX_CANDIDATES
    ids = torch.from_numpy(sampler.request_ids(2, n)).cuda()
    out = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = small.ctx.lib.aif_score(small.ctx.h, st2.handle, C.c_void_p(ids.data_ptr()), n, C.c_void_p(out.data_ptr()), stream)
    assert rc == B.ERR_SHAPE
    rc = small.ctx.lib.aif_score_noalloc(small.ctx.h, st2.handle, C.c_void_p(ids.data_ptr()), n, C.c_void_p(out.data_ptr()), stream)
    assert rc == B.OK, small.ctx.lib.aif_last_error().decode()
    torch.cuda.synchronize()
    want = oracle.score(table, oreq, ids.cpu().numpy())
    assert np.abs(out.cpu().numpy() - want).max() <= TOL
    assert small.ctx.poll_status() == 0
    small.close()
