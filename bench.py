#!/usr/bin/env python
"""Benchmark of the AIF pre-ranking scoring pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

One "step" is one pass of the whole real-time path (gather, interaction blocks, scoring MLP) over one batch of
synthetic candidates: one aif_score call on a 10^4-candidate request for the default workload (the paper-shaped
single request), one aif_score_batch call for the multi-request workloads.  User states are computed beforehand by
aif_user_precompute (they belong to the retrieval phase, not to the timed real-time phase).

Prints ONE JSON line (rank 0).  `value` is candidates scored per second with ids already resident in GPU memory;
`e2e` is the same metric through aif_score_host with host buffers (H2D of the ids and D2H of the logits inside the
timed region).  With --gpus N > 1 (launched by torchrun) every rank runs an independent replica on its own GPU:
the path does not shard, so there is no data-path collective; the time is the max over ranks.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2511_12934_b200 import synth

METRIC = "candidates scored/s (p50 latency per request reported beside it), 1 B200"
UNIT = "candidates/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # CUDA-core kernels: SMs x lanes x 2 x max clock
NOMINAL_BF16_TFLOPS = 2250.0                               # dense bf16, the data-sheet figure
NOMINAL_HBM_GBS = 8000.0


def ncu_traffic_table():
    """DRAM read + write bytes of the scoring kernels as ncu counted them: {(workload, kernel): (unit, bytes)} with unit
    "per_launch" (captured on the benchmark's own workload) or "per_candidate" (captured on a scaled copy of it; the
    traffic of these kernels grows with the candidates).  The table is a text file kept beside the ncu summaries."""
    out = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return out
    with open(path) as fh:
        for ln in fh:
            parts = ln.split()
            if len(parts) == 4 and not ln.startswith("#"):
                out[(parts[0], parts[1])] = (parts[2], float(parts[3]))
    return out


# ----------------------------------------------------------------------------------------------------------------
# algorithmic work (what the method itself has to do; padding and recomputation are not counted)
# ----------------------------------------------------------------------------------------------------------------
def flops_per_candidate(wl: synth.Workload, keys=None) -> dict:
    """keys: mean number of sequence items a candidate interacts with (the whole sequence unless the workload has
    category sub-sequences)."""
    k1 = wl.input_width() - wl.d                       # the user columns are done once per request
    keys = float(wl.L if keys is None else keys)
    f = {"attention": 4.0 * keys * wl.d if wl.blocks & synth.BLK_ATT else 0.0}
    f["lsh_din"] = 2.0 * keys * wl.d if wl.blocks & synth.BLK_LSH_DIN else 0.0
    f["bea"] = 2.0 * wl.n_bridge * wl.d if wl.blocks & synth.BLK_BEA else 0.0
    widths = [k1] + list(wl.hidden)
    for i in range(len(wl.hidden)):
        f[f"layer{i + 1}"] = 2.0 * widths[i] * widths[i + 1]
    f[f"layer{len(wl.hidden)}"] += 2.0 * wl.hidden[-1]  # output dot rides in the last hidden layer's kernel
    f["total"] = sum(f.values())
    return f


def kernel_flops(name: str, wl: synth.Workload, n: int, keys=None) -> float:
    f = flops_per_candidate(wl, keys)
    if name in ("score_simt", "score_fused"):
        return f["total"] * n
    if name == "interact":
        return (f["attention"] + f["lsh_din"] + f["bea"]) * n
    if name == "lsh":          # eq. 8's contraction; the match counts of eqs. 6-7 ride in the same kernel (see lsh_note)
        return f["lsh_din"] * n
    if name in ("buckets", "group"):
        return 0.0
    return f.get(name, 0.0) * n


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            return json.load(fh), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])), mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------------------------
# the oracle legs (CPU): cpu_baseline and --impl reference
# ----------------------------------------------------------------------------------------------------------------
def oracle_setup(wl):
    from oracle import aif_oracle as orc
    from tests import helpers
    weights = synth.make_weights(wl)
    table = synth.make_item_table(wl)
    oracle = helpers.make_oracle(wl, weights, M=table["E"].shape[0])
    rq = synth.make_request(wl, 0)
    ids = synth.IdSampler(wl).request_ids(0)
    return oracle, table, helpers.projected_request(wl, rq), ids, orc.num_threads()


def oracle_sample_size(wl, core_seconds=12.0):
    # the scalar fp64 oracle sustains roughly 1 GFLOP/s per core
    n = int(core_seconds * 1.0e9 / flops_per_candidate(wl)["total"])
    return max(32, min(wl.N, n))


def cpu_baseline(wl, pre=None):
    oracle, table, req, ids, threads = pre or oracle_setup(wl)
    n = oracle_sample_size(wl)
    # repeat the sample until about 12 core-seconds of oracle work have been timed
    passes, dt = 0, 0.0
    while passes == 0 or (dt * threads < 12.0 and passes < 64):
        t0 = time.perf_counter()
        oracle.score(table, req, ids[:n])
        dt += time.perf_counter() - t0
        passes += 1
    return {"value": n * passes / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {n} candidates of request 0 of {wl.name}, scored {passes} times ({dt:.2f} s wall)",
            "ms_per_1e4_candidates": 1e4 * dt / (n * passes) * 1e3}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pre = oracle_setup(wl)
    oracle, table, req, ids, threads = pre
    # size the per-step sample so that warm-up + K steps end within about two minutes on this host
    per_step_core_s = min(4.0, 110.0 * threads / max(1, args.steps + args.warmup))
    n = max(32, oracle_sample_size(wl, core_seconds=per_step_core_s))
    for _ in range(args.warmup):
        oracle.score(table, req, ids[:n])
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        oracle.score(table, req, ids[:n])
        times.append(time.perf_counter() - t0)
    total = sum(times)
    value = n * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "candidates_per_step": n, "note": "CPU oracle, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"first {n} candidates of request 0 of {wl.name} per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------------------------
def replica_plan(world: int, rank: int) -> dict:
    """Multi-GPU plan: the path does not shard, every rank is an independent replica of the whole workload."""
    return {"rank": rank, "world": world, "replica": True, "share_of_work": 1.0}


def reduce_max(value: float, dist=None) -> float:
    """Max over ranks of a scalar (device-side when NCCL is the backend)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args, wl):
    import torch
    from paper_2511_12934_b200 import build as libbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    libbuild.build()
    line = measure(args, wl, args.steps, args.warmup, dist, world, rank, full=True)
    if world == 1 and args.also:
        # the other bf16 shapes of the benchmark definition, briefly, so that one run shows every roofline fraction
        others = {}
        for name in args.also.split(","):
            o = measure(args, synth.SHORT[name], 20, 3, None, 1, 0, full=False)
            others[name] = {k: o[k] for k in ("value", "unit", "ms_per_step", "p50_ms_per_request", "p99_ms_per_request",
                                              "latency_samples", "flops_per_candidate", "config", "roofline", "step_tflops",
                                              "step_frac", "e2e")}
        line["other_workloads"] = others
    if rank == 0 and world == 1 and args.bea_sweep and wl.dtype == "bf16":
        line["bea_bridge_sweep"] = bea_sweep(wl)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def bea_sweep(base: synth.Workload, bridges=(1, 2, 4, 8, 16), m_features=64, steps=30):
    """Cost of Bridge Embedding Approximation over the number of bridges n (Algorithm 1; Section 5.2.2 studies quality over
    n, this is the cost side): the user-side call that computes W = Softmax(B U^T / sqrt(d)) and V from m_features user
    feature embeddings, and the scoring step with the BEA block on (v = w_hat V per candidate, d more input columns)."""
    import torch
    from paper_2511_12934_b200 import binding as B
    from paper_2511_12934_b200 import serving
    out = []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for n in bridges:
        wl = base.with_(name=f"{base.name}_bea{n}", M=min(base.M, 200_000), blocks=base.blocks | synth.BLK_BEA, n_bridge=n)
        weights, table = synth.make_weights(wl), synth.make_item_table(wl)
        srv = serving.Server(wl, weights, table, max_user_states=2, max_batch_candidates=wl.N)
        rq = synth.make_request(wl, 0)
        rq = dict(rq, bea_U=synth.normal_rows(m_features, wl.d, 1.0, wl.dtype, 77, n))
        del rq["V"]
        dev = srv.upload_request(rq, B.USER_PROJECTED)
        ids = torch.from_numpy(synth.IdSampler(wl).request_ids(0)).cuda()
        logits = torch.empty(wl.N, dtype=torch.float32, device="cuda")
        st = srv.precompute(0, dev)
        torch.cuda.synchronize()
        pre, sc = [], []
        for i in range(steps):
            a, b, c, d = (torch.cuda.Event(enable_timing=True) for _ in range(4))
            st.release()
            a.record(srv.side)
            st = srv.precompute(1 + i, dev)
            b.record(srv.side)
            torch.cuda.synchronize()
            flush.zero_()
            c.record()
            srv.ctx.score(st, ids, logits)
            d.record()
            torch.cuda.synchronize()
            pre.append(a.elapsed_time(b)), sc.append(c.elapsed_time(d))
        out.append({"n_bridge": n, "user_side_ms": float(np.median(pre[3:])), "score_ms": float(np.median(sc[3:])),
                    "candidates": wl.N, "m_features": m_features})
        srv.close()
        del srv
    return out


def measure(args, wl, steps, warmup, dist, world, rank, full):
    """Times `steps` scoring steps of one workload on this rank's GPU; returns the JSON line as a dict."""
    import torch
    from paper_2511_12934_b200 import binding as B
    from paper_2511_12934_b200 import serving

    plan = replica_plan(world, rank)
    path = {"auto": B.PATH_AUTO, "simt": B.PATH_SIMT, "tensor": B.PATH_TENSOR}[args.path]
    weights = synth.make_weights(wl)
    table = synth.make_item_table(wl)
    batch = wl.R > 1
    pool = 1 if batch else 8                      # distinct requests cycled over the steps (single-request workload)
    n_states = wl.R if batch else pool
    srv = serving.Server(wl, weights, table, path=path, max_user_states=n_states,
                         max_batch_candidates=wl.R * wl.N if batch else wl.N)
    sampler = synth.IdSampler(wl)
    states, id_lists = [], []
    key_sum = 0.0
    for r in range(n_states):
        rq = synth.make_request(wl, r)
        states.append(srv.precompute(r, srv.upload_request(rq, B.USER_PROJECTED)))
        id_lists.append(sampler.request_ids(r))
        if wl.n_categories:   # sequence items each candidate meets: the length of its category's sub-sequence
            lens = np.bincount(rq["seq_cat"], minlength=wl.n_categories)
            cats = np.array([srv.ctx.lib.aif_category(int(i), wl.n_categories, wl.bucket_mode) for i in id_lists[-1]])
            key_sum += float(lens[cats].sum())
    keys = key_sum / sum(len(x) for x in id_lists) if wl.n_categories else None
    torch.cuda.synchronize()
    if batch:
        offs = np.zeros(wl.R + 1, dtype=np.int64)
        offs[1:] = np.cumsum([len(x) for x in id_lists])
        ids_dev = [torch.from_numpy(np.concatenate(id_lists)).cuda()]
        cands = int(offs[-1])
    else:
        ids_dev = [torch.from_numpy(x).cuda() for x in id_lists]
        cands = wl.N
    logits = torch.empty(cands, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > L2 (126 MB)

    def step(i):
        if batch:
            srv.ctx.score_batch(states, ids_dev[0], offs, logits)
        else:
            srv.ctx.score(states[i % pool], ids_dev[i % pool], logits)

    def timed(n_steps, fn):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_steps)]
        for i in range(n_steps):
            flush.zero_()
            ev[i][0].record()
            fn(i)
            ev[i][1].record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    # the clock sampler starts before the warm-up so that it is running when the timed region begins; it stops after the
    # latency pass
    uuid = str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
    sampler_proc = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    time.sleep(0.4)
    for i in range(max(3, warmup)):
        flush.zero_()
        step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = B.kernel_launches()
    times = timed(steps, step)
    launches = B.kernel_launches() - launches0
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    total_ms = reduce_max(sum(times), dist)

    # end to end: host ids in, host logits out, through aif_score_host (one call per request)
    if batch:
        host_ids = [torch.from_numpy(np.concatenate(id_lists)).pin_memory()]
        host_out = [torch.empty(cands, dtype=torch.float32).pin_memory()]
    else:
        host_ids = [torch.from_numpy(x).pin_memory() for x in id_lists]
        host_out = [torch.empty(len(x), dtype=torch.float32).pin_memory() for x in id_lists]

    def step_e2e(i):
        if batch:
            srv.ctx.score_batch_host(states, host_ids[0], offs, host_out[0])
        else:
            srv.ctx.score_host(states[i % pool], host_ids[i % pool], host_out[i % pool])

    e2e_steps = max(3, min(steps, 50)) if full else 3
    step_e2e(0)
    e2e_times = timed(e2e_steps, step_e2e)
    e2e_ms = reduce_max(sum(e2e_times), dist)

    # per-request latency percentiles from a pass of their own, whatever --steps says: one sample per scoring call
    # (a launch over R requests gives its time divided by R), L2 flushed before each
    lat_calls = (1000 if full else 100) if not batch else max(20, min(1000 if full else 60, int(4000.0 / max(1e-3, float(np.mean(times))))))
    if args.latency_calls >= 0:
        lat_calls = max(2, args.latency_calls)
    lat_times = timed(lat_calls, step)
    clocks = sampler_proc.stop()

    # per-kernel durations (events inside the library), for the roofline of the dominant kernel
    srv.ctx.set_kernel_timing(True)
    ksum, kcount = {}, 0
    for i in range(min(steps, 50)):
        flush.zero_()
        step(i)
        for k, v in srv.ctx.get_kernel_timing().items():
            ksum[k] = ksum.get(k, 0.0) + v
        kcount += 1
    srv.ctx.set_kernel_timing(False)
    kavg = {k: v / kcount for k, v in ksum.items()}
    assert srv.ctx.poll_status() == 0, "device status word set during the benchmark"

    # the gather stage alone (aif_gather_rows) on a long id stream drawn like the workload's candidates: HBM roofline
    gn = 1 << 22
    g_ids = torch.from_numpy(sampler._raw(np.random.default_rng(7), gn).astype(np.int32)).cuda()
    g_out = torch.empty(gn, wl.d, dtype=torch.float32 if wl.dtype == "f32" else torch.bfloat16, device="cuda")
    row_bytes = wl.d * (4 if wl.dtype == "f32" else 2)

    def gather_step(i):
        srv.ctx.gather_rows(g_ids, g_out)

    gather_step(0)
    g_ms = float(np.median(timed(10, gather_step)))
    # the same over distinct rows (a seeded permutation of the table, at most 2^22 of them): no row is read twice, so L2
    # cannot serve repeats and the figure is an HBM figure (the table is larger than L2 for every bf16 workload)
    gd = int(min(gn, table["E"].shape[0]))
    d_ids = torch.from_numpy(np.random.default_rng(8).permutation(table["E"].shape[0])[:gd].astype(np.int32)).cuda()

    def gather_distinct(i):
        srv.ctx.gather_rows(d_ids, g_out[:gd])

    gather_distinct(0)
    gd_ms = float(np.median(timed(10, gather_distinct)))
    del g_out, d_ids

    # the user-side call (eqs. 1-3 from raw embeddings + pre-cache + p_u) on the side stream: the time a retrieval phase has
    # to cover; one extra arena slot is not available, so a state of the pool is recomputed in place of itself
    pre_ms, overlap = None, None
    if full:
        states[-1].release()
        dev_raw = srv.upload_request(synth.make_request(wl, n_states - 1), B.USER_RAW)
        ts = []
        for i in range(6):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(srv.side)
            stx = srv.precompute(10_000 + i, dev_raw)
            b.record(srv.side)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
            if i < 5:
                stx.release()
        pre_ms = float(np.median(ts[1:]))
        # Overlap with a simulated retrieval phase (Section 3.1: the user side runs while the candidates are retrieved): the
        # main stream is busy for `retrieval_ms` (a spin kernel standing in for the retrieval service), the user-side call
        # runs on the side stream from the same starting point, scoring follows on the main stream and waits for both.  All
        # times from events: the request takes retrieval + scoring, not retrieval + precompute + scoring.
        stx.release()
        hz = 1e3 * torch.cuda.get_device_properties(torch.cuda.current_device()).clock_rate   # kHz -> Hz
        retrieval_cycles = int(max(3.0 * pre_ms, 0.3) * 1e-3 * hz)
        ids_o = ids_dev[0] if batch else ids_dev[(n_states - 1) % pool]
        main = torch.cuda.current_stream()
        rows = []
        for i in range(8):
            e0, e_ret, e_end = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            e0.record(main)
            srv.side.wait_event(e0)
            torch.cuda._sleep(retrieval_cycles)
            e_ret.record(main)
            s0.record(srv.side)
            stx = srv.precompute(20_000 + i, dev_raw)
            s1.record(srv.side)
            if batch:
                srv.ctx.score_batch(states[:-1] + [stx], ids_o, offs, logits)
            else:
                srv.ctx.score(stx, ids_o, logits)
            e_end.record(main)
            torch.cuda.synchronize()
            rows.append((e0.elapsed_time(e_ret), e0.elapsed_time(s1), e_ret.elapsed_time(e_end), e0.elapsed_time(e_end)))
            if i < 7:
                stx.release()
        states[-1] = stx
        r = np.median(np.array(rows[1:]), axis=0)
        overlap = {"retrieval_ms": float(r[0]), "precompute_done_ms_after_start": float(r[1]), "scoring_ms_after_retrieval": float(r[2]),
                   "request_ms": float(r[3]), "sum_if_serial_ms": float(r[0] + pre_ms + r[2]),
                   "hidden": bool(r[1] <= r[0]), "note": "medians of 7 runs; retrieval = a spin kernel on the main stream"}

    # the item side of the nearline pipeline as a compute call (eq. 4 tower; bridge weights and signatures when their
    # blocks are on): 2^19 synthetic items with dI = 4 d, hI = 2 d written into the table rows they will be gathered from
    nearline = None
    if full and rank == 0 and not wl.blocks & (synth.BLK_BEA | synth.BLK_LSH_DIN | synth.BLK_SIMTIER):
        nn = int(min(1 << 19, table["E"].shape[0]))
        it = synth.make_item_side(wl, nn)
        bdt = B.F32 if wl.dtype == "f32" else B.BF16
        dev_it = {k: (torch.from_numpy(v).cuda() if v.dtype == np.float32 else B.to_device(v, bdt)) for k, v in it.items()}
        saved = torch.empty(nn, wl.d, dtype=torch.float32 if wl.dtype == "f32" else torch.bfloat16, device="cuda")
        srv.ctx.gather_rows(torch.arange(nn, dtype=torch.int32, device="cuda"), saved)   # the table is put back afterwards
        srv.ctx.load_item_weights(dev_it)

        def nearline_step(i):
            srv.ctx.item_nearline_compute(None, dev_it["I_raw"], dev_it["I_id"], dev_it["M_mm"])

        nearline_step(0)
        n_ms = float(np.median(timed(5, nearline_step)))
        dI, hI = it["W_i0"].shape[1], it["W_i0"].shape[0]
        n_flops = 2.0 * (dI * hI + hI * wl.d)
        el = 4 if wl.dtype == "f32" else 2
        nearline = {"items": nn, "dI": dI, "hI": hI, "ms": n_ms, "items_per_s": nn / (n_ms * 1e-3),
                    "tflops": nn * n_flops / (n_ms * 1e-3) / 1e12, "gbs": nn * (dI + wl.d) * el / (n_ms * 1e-3) / 1e9,
                    "note": "tower flops and (raw row in + item vector out) bytes; one kernel, hidden activations in tensor memory"}
        srv.ctx.item_nearline_refresh(None, saved)
        del dev_it, saved

    peaks, peak_kind = load_peaks()
    gather = {"rows": gd, "row_bytes": row_bytes, "ms": gd_ms, "achieved": gd * (2 * row_bytes + 4) / (gd_ms * 1e-3) / 1e9,
              "peak": float(peaks["hbm_gbs"]), "unit": "GB/s", "bound": "hbm", "peak_kind": f"copy bandwidth, {peak_kind}",
              "ids": "distinct rows (seeded permutation of the table): every row comes from HBM once",
              "table_bytes": int(table["E"].shape[0]) * row_bytes}
    gather["frac"] = gather["achieved"] / gather["peak"]
    gather["frac_nominal"] = gather["achieved"] / NOMINAL_HBM_GBS
    rep_gbs = gn * (2 * row_bytes + 4) / (g_ms * 1e-3) / 1e9
    gather["with_repeats"] = {"rows": gn, "ms": g_ms, "achieved": rep_gbs, "frac": rep_gbs / float(peaks["hbm_gbs"]),
                              "ids": "drawn like the workload's candidates (Zipf), repeats allowed: hot rows are served by L2"}
    gt = ncu_traffic_table().get(("gather_stage", "k_gather_rows"))
    gather["traffic"] = None if gt is None else int(gt[1] * (gd if gt[0] == "per_candidate" else 1))
    top = max(kavg, key=kavg.get)
    tensor = bool(srv.ctx.get_stats().tensor_path) and top != "interact"
    kf = kernel_flops(top, wl, cands, keys)
    if tensor:
        peak = float(peaks["bf16_tflops"])
        roof = {"bound": "tensor", "kernel": top, "achieved": kf / (kavg[top] * 1e-3) / 1e12, "peak": peak,
                "unit": "TFLOP/s", "peak_kind": f"bf16 burst, {peak_kind}"}
    else:
        roof = {"bound": "alu", "kernel": top, "achieved": kf / (kavg[top] * 1e-3) / 1e12, "peak": FP32_FMA_PEAK_TFLOPS,
                "unit": "TFLOP/s", "peak_kind": "fp32 FMA: 148 SMs x 128 lanes x 2 x 1.965 GHz"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    if top == "lsh":
        roof["lsh_note"] = (f"eqs. 6-7 need {wl.lsh_bits // 32} xor + popc on 32-bit words per (candidate, key) pair by the definition; "
                            f"the kernel gets the counts from a +-1 fp8 product ({2 * wl.lsh_bits} tensor flop per pair, not counted "
                            "in `achieved`) and spends about ten integer / fp32 instructions per pair on conversion and tiers")
    if tensor:
        roof["frac_nominal"] = roof["achieved"] / NOMINAL_BF16_TFLOPS
        roof["peak_nominal"] = NOMINAL_BF16_TFLOPS
    traffic = ncu_traffic_table().get((wl.name, top))
    roof["traffic"] = None if traffic is None else int(traffic[1] * (cands if traffic[0] == "per_candidate" else 1))
    roof["traffic_source"] = None if traffic is None else f"ncu dram bytes read + write, {traffic[0].replace('_', ' ')}"
    roof["kernel_ms"] = kavg

    value = world * cands * steps / (total_ms * 1e-3)
    per_request_ms = [t / (wl.R if batch else 1) for t in lat_times]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": max(3, warmup),
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": wl.name, "requests_per_step": wl.R, "candidates_per_step": cands, "M": wl.M, "d": wl.d,
                   "L": wl.L, "F": wl.F, "hidden": list(wl.hidden), "mini_batch": wl.mini_batch,
                   "l2": "flushed between timed steps (256 MiB memset)", "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "path": "tensor" if srv.ctx.get_stats().tensor_path else "cuda-core",
                   "request_pool": pool, "n_categories": wl.n_categories,
                   "mean_keys_per_candidate": keys if keys is not None else wl.L},
        "p50_ms_per_request": float(np.percentile(per_request_ms, 50)),
        "p99_ms_per_request": float(np.percentile(per_request_ms, 99)),
        "latency_samples": {"scoring_calls": len(lat_times), "requests_per_call": wl.R if batch else 1},
        "flops_per_candidate": flops_per_candidate(wl, keys)["total"],
        "step_tflops": flops_per_candidate(wl, keys)["total"] * cands * steps / (total_ms * 1e-3) / 1e12,
        "step_frac": {"of_measured_peak": flops_per_candidate(wl, keys)["total"] * cands * steps / (total_ms * 1e-3) / 1e12 / float(peaks["bf16_tflops"]),
                      "of_nominal_peak": flops_per_candidate(wl, keys)["total"] * cands * steps / (total_ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS}
        if wl.dtype == "bf16" else None,
        "e2e": {"value": world * cands * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * cands,
                "d2h_bytes_per_step": 4 * cands, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roof,
        "gather_stage": gather,
        "nearline_item_side": nearline,
        "user_precompute": {"ms": pre_ms, "inputs": "raw embeddings (eqs. 1-3 computed)", "L": wl.L, "stream": "side", "overlap": overlap},
        "replica_plan": plan,
    }
    srv.close()
    del srv, flush, logits, ids_dev, g_ids
    torch.cuda.empty_cache()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(synth.SHORT))
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-bea-sweep", dest="bea_sweep", action="store_false", help="skip the cost table over the number of BEA bridges")
    ap.add_argument("--also", default="c3,c4,c4_lsh,c4_both,long_lsh,long_sim,c5", help="other workloads measured briefly after the main one ('' = none)")
    # scaled copies of a workload, for profiler captures that must stay small (the defaults are the full sizes)
    ap.add_argument("--latency-calls", type=int, default=-1, help="scoring calls of the latency pass (default: 1000, fewer for long steps)")
    ap.add_argument("--requests", type=int, default=0, help="override the number of requests per step")
    ap.add_argument("--rows", type=int, default=0, help="override the rows of the item table")
    args = ap.parse_args()
    wl = synth.SHORT[args.workload]
    if args.requests:
        wl = wl.with_(R=args.requests)
    if args.rows:
        wl = wl.with_(M=args.rows)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
