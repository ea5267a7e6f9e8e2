#!/usr/bin/env python
"""Benchmark of the trimmed-vocabulary draft head on B200.

One step = one ``vt_draft_head`` call (contraction, top-k, log-softmax, d2t remap: one launch) on the
workload ``d=4096, V_trim=32000 of V_full=128256, M=8, k=8``.  The once-per-model steps (head
compaction, coverage of the token stream) are timed separately and reported under ``once_per_model``.
Inputs are synthetic and seeded.  Successive calls rotate over enough copies of ``W_trim`` that every
call streams its weights from HBM rather than from L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-curve]

prints one JSON line (rank 0).  ``--impl reference`` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_05210_b200 import inputs  # noqa: E402

METRIC = "draft_head_us_per_call"
UNIT = "us/call"
WORKLOAD = dict(d=4096, V_full=inputs.V_LLAMA3, V_trim=32000, M=8, k=8, seed=3000)
WORKLOAD_NAME = "d=4096, V_trim=32000 of V_full=128256, M=8, top-k=8, log-softmax over V_trim, d2t remap"
CURVE_VT = (4096, 4380, 6521, 8192, 13264, 16384, 32000, 128256)   # incl. the paper's vocabulary sizes (Sections 2.6, 3.2)
REPS = 5              # repetitions of the timed region (median, spread and a 95 % interval are reported)
ISOLATED_CALLS = 200  # single calls timed one by one behind an unrelated kernel
CURVE_M = (1, 2, 4, 8, 16, 32, 64)
FALLBACK_HBM_GBS = 6650.0


def head_bytes(d, Vt, M, k):
    """Algorithmic bytes of one call: weights once, hidden states, d2t gathers and both outputs."""
    return 2 * d * Vt + 2 * M * d + M * k * 12


# DRAM traffic of one head launch on the bench workload from the ncu capture summarised in
# profiles/head_mma_small_d4096_vt32000_m8.md (dram__bytes_read.sum + dram__bytes_write.sum), valid while the
# kernel sources still hash to the value recorded there.
NCU_TRAFFIC = {"bytes": 264_363_520 + 4_110_080, "source_hash": "ac01381d7e9f9884",
               "sources": ("paper_2603_05210_b200/csrc/vt_head_mma_small.cu", "paper_2603_05210_b200/csrc/vt_common.cuh",
                           "paper_2603_05210_b200/csrc/vt_tc.cuh")}


def ncu_traffic_or_none():
    import hashlib
    h = hashlib.sha256()
    try:
        for rel in NCU_TRAFFIC["sources"]:
            with open(os.path.join(ROOT, rel), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    return NCU_TRAFFIC["bytes"] if h.hexdigest()[:16] == NCU_TRAFFIC["source_hash"] else None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(x: float, dist, device) -> float:
    """The slowest rank's figure: every multi-GPU number is the max over ranks."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_call(us_per_call_slowest_rank: float, world: int) -> float:
    """N replicas each finish one call in that time: the job's time per call is 1/N of it (weak scaling)."""
    return us_per_call_slowest_rank / world


def to_dev(a, torch, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.view(dtype) if dtype is not None else t


GRAPH_CALLS = 120     # calls per captured CUDA graph (a multiple of every copy count the bench uses: 2..6, 8, 10, 12...)


def stats(xs):
    """median, 10th / 90th percentile and the 95 % interval of the mean of a list of samples."""
    a = np.asarray(xs, dtype=np.float64)
    half = 1.96 * float(a.std(ddof=1)) / np.sqrt(a.size) if a.size > 1 else 0.0
    return {"median": round(float(np.median(a)), 3), "p10": round(float(np.percentile(a, 10)), 3),
            "p90": round(float(np.percentile(a, 90)), 3), "mean": round(float(a.mean()), 3),
            "ci95": [round(float(a.mean()) - half, 3), round(float(a.mean()) + half, 3)], "n": int(a.size)}


def time_head(vt, torch, h, W_copies, d2t, k, steps, warmup, path=0, use_graph=True, reps=1, static_weights=False):
    """CUDA-event times of `reps` regions of exactly `steps` back-to-back calls rotating over W_copies.

    Returns (ms of the first region if reps == 1 else the list of ms per region, launches per call).
    With use_graph the calls are replayed from a captured CUDA graph of GRAPH_CALLS calls (plus directly
    launched calls for the remainder), the way a serving loop would issue them; otherwise every call goes
    through the Python binding.  Either way each call is a separate kernel launch on the stream.
    """
    M = h.shape[0]
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, k))
    tid = torch.empty((M, k), dtype=torch.int32, device="cuda")
    lp = torch.empty((M, k), dtype=torch.float32, device="cuda")
    n = len(W_copies)

    def call(i):
        vt.vt_draft_head(h, W_copies[i % n], d2t, k, workspace=ws, path=path, target_ids=tid, logprobs=lp,
                         static_weights=static_weights)

    for i in range(warmup):
        call(i)
    launches = vt.vt_last_launch_count()
    graph = None
    n_replay = steps // GRAPH_CALLS if use_graph else 0
    if n_replay > 0:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(GRAPH_CALLS):
                    call(i)
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()                                   # one untimed replay: graph upload
    out = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_replay):
            graph.replay()
        for i in range(steps - n_replay * GRAPH_CALLS):
            call(i)
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1))
    assert vt.vt_last_status(ws) == vt.VT_OK, "a device-side wait ran out during the timed region"
    return (out[0] if reps == 1 else out), launches


def hold_gpu(torch, ms=8.0):
    """Keeps the stream busy for a few milliseconds so that the host can enqueue what follows without the GPU ever
    waiting for it: what is timed afterwards is device time, not the host's launch overhead."""
    torch.cuda._sleep(int(ms * 1e-3 * 1.9e9))


def time_isolated(vt, torch, h, W_copies, d2t, k, n_calls=ISOLATED_CALLS, path=0):
    """us of ONE call that follows an unrelated, ordinary kernel (an elementwise update of a 32 MB tensor: no
    programmatic early trigger, and it displaces part of L2), timed with a CUDA event pair per call on a cold
    copy of W_trim; the list of n_calls samples.  This is what a draft step sees inside a serving loop, where
    the head follows the decoder layer and not another head call."""
    M = h.shape[0]
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, k))
    tid = torch.empty((M, k), dtype=torch.int32, device="cuda")
    lp = torch.empty((M, k), dtype=torch.float32, device="cuda")
    filler = torch.zeros(8 << 20, dtype=torch.float32, device="cuda")
    n = len(W_copies)
    for i in range(5):
        vt.vt_draft_head(h, W_copies[i % n], d2t, k, workspace=ws, path=path, target_ids=tid, logprobs=lp)
    pairs = []
    torch.cuda.synchronize()
    hold_gpu(torch)          # the host enqueues all samples while the GPU is held, so no sample waits for the host
    for i in range(n_calls):
        filler.add_(1.0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        vt.vt_draft_head(h, W_copies[i % n], d2t, k, workspace=ws, path=path, target_ids=tid, logprobs=lp)
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    assert vt.vt_last_status(ws) == vt.VT_OK
    return [a.elapsed_time(b) * 1000.0 for a, b in pairs]


def n_copies_for_cold(bytes_per_copy, l2_bytes, free_bytes):
    want = max(2, -(-4 * l2_bytes // bytes_per_copy))
    return int(max(1, min(want, (free_bytes // 2) // bytes_per_copy)))


def run_ours(args):
    import torch

    import paper_2603_05210_b200 as vt

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the draft head")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    vt.lib()
    props = torch.cuda.get_device_properties(local)
    l2 = int(props.L2_cache_size)
    peak_gbs, peak_kind = measured_peaks()

    w = WORKLOAD
    d, V, Vt, M, k = w["d"], w["V_full"], w["V_trim"], w["M"], w["k"]
    if args.m is not None:      # another draft-row count on the same weights (profiling the other head kernels)
        M = args.m
    tokens = inputs.zipf_token_stream(V, 1.1, 1_000_000, w["seed"])
    ranking = inputs.frequency_ranking(tokens, V)
    case = inputs.make_case("bench", d, Vt, M, k, w["seed"], row_scale=(0.5, 2.0), ranking=ranking)
    W_full = to_dev(case.W_full.view(np.int16), torch, torch.bfloat16)
    keep = to_dev(case.keep_ids, torch)
    d2t = to_dev(case.d2t, torch)
    h = to_dev(case.h.view(np.int16), torch, torch.bfloat16)
    tok_dev = to_dev(tokens, torch)

    # once-per-model steps: compaction (a1), coverage (a6), vocabulary selection
    W_trim = vt.vt_compact_head(W_full, keep)
    once = once_per_model(vt, torch, W_full, keep, W_trim, tok_dev, tokens, d, V, peak_gbs) if rank == 0 else {}

    free, _ = torch.cuda.mem_get_info()
    nc = n_copies_for_cold(W_trim.numel() * 2, l2, free)
    copies = [W_trim] + [W_trim.clone() for _ in range(nc - 1)]

    # ---- timed region: REPS x K calls, device-timed, max over ranks; the headline is the median region
    sampler = ClockSampler(local)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ms_list, launches_per_call = time_head(vt, torch, h, copies, d2t, k, args.steps, args.warmup,
                                           use_graph=not args.no_graph, reps=REPS)
    clocks = sampler.stop()
    ms_list = [max_over_ranks(x, dist, "cuda") for x in ms_list]
    if dist is not None:
        dist.barrier()
    us_list = [x * 1000.0 / args.steps for x in ms_list]
    us_per_call_rank = float(np.median(us_list))
    ms = us_per_call_rank * args.steps / 1000.0
    value = whole_job_us_per_call(us_per_call_rank, world)
    bytes_call = head_bytes(d, Vt, M, k)
    achieved = bytes_call / (us_per_call_rank * 1e-6) / 1e9

    # the same region with W_trim declared constant (VT_HEAD_STATIC_WEIGHTS): weights requested ahead of the
    # stream-order wait; and single calls behind an unrelated kernel (what a serving loop sees)
    ms_static, _ = time_head(vt, torch, h, copies, d2t, k, args.steps, min(args.warmup, 50), use_graph=not args.no_graph,
                             reps=REPS, static_weights=True)
    us_static = float(np.median([max_over_ranks(x, dist, "cuda") for x in ms_static])) * 1000.0 / args.steps
    iso = time_isolated(vt, torch, h, copies, d2t, k)
    us_iso = max_over_ranks(float(np.median(iso)), dist, "cuda")

    # ---- end to end: host h -> device, head, outputs -> host, every step
    e2e_steps = max(1, min(args.steps, 2000))
    hws = vt.new_workspace(vt.vt_host_workspace_bytes(M, d, k))
    h_host = torch.from_numpy(case.h.view(np.int16).copy()).pin_memory()
    tid_h = torch.empty((M, k), dtype=torch.int32).pin_memory()
    lp_h = torch.empty((M, k), dtype=torch.float32).pin_memory()
    # the C entry point itself, with the pointers resolved once (what a C or C++ caller does every step)
    c_call = vt.lib().vt_draft_head_host
    w_ptrs = [w_.data_ptr() for w_ in copies]
    fixed_args = (d2t.data_ptr(), M, d, Vt, k, tid_h.data_ptr(), lp_h.data_ptr(), hws.data_ptr(), hws.numel(),
                  torch.cuda.current_stream().cuda_stream)
    for i in range(min(args.warmup, 50)):
        assert c_call(h_host.data_ptr(), w_ptrs[i % nc], *fixed_args) == vt.VT_OK
    torch.cuda.synchronize()
    h_ptr = h_host.data_ptr()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        c_call(h_ptr, w_ptrs[i % nc], *fixed_args)
    e2e_us = (time.perf_counter() - t0) * 1e6 / e2e_steps
    assert vt.vt_last_status(hws) == vt.VT_OK
    e2e_us = max_over_ranks(e2e_us, dist, "cuda")

    line = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 6), "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in, fp32 accumulate", "data": "synthetic",
        "config": bench_config(WORKLOAD_NAME if args.m is None else WORKLOAD_NAME.replace("M=8", f"M={M}"),
                               cold=f"calls rotate over {nc} copies of W_trim ({nc * W_trim.numel() * 2 / 1e6:.0f} MB >= 4x L2 of "
                                    f"{l2 / 1e6:.0f} MB): inputs larger than L2",
                               step="one vt_draft_head call (contraction + top-k + log-softmax + remap, one launch), default options",
                               launch="eager calls through the binding" if args.no_graph or args.steps < GRAPH_CALLS
                               else f"CUDA-graph replay of {GRAPH_CALLS}-call graphs (one kernel launch per call)",
                               parallelism="replicas only" if world > 1 else "single GPU",
                               calls_per_s=round(1e6 / value, 1)),
        "repetitions": {"regions": REPS, "us_per_call": stats(us_list), "value_is": "median region"},
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak_gbs, "unit": "GB/s",
                     "frac": round(achieved / peak_gbs, 4), "of": peak_kind, "traffic": None if args.m is not None else ncu_traffic_or_none(),
                     "algorithmic_bytes_per_launch": bytes_call, "frac_of_nominal_8TBs": round(achieved / 8000.0, 4),
                     "frac_isolated": round(bytes_call / (us_iso * 1e-6) / 1e9 / peak_gbs, 4),
                     "frac_static_weights": round(bytes_call / (us_static * 1e-6) / 1e9 / peak_gbs, 4),
                     "kernel": "head kernel of the chosen path; duration = timed region / launches (back-to-back calls); "
                               "frac_isolated = the same bytes over the single-call latency below"},
        "isolated_call": {"us": stats(iso), "calls": len(iso),
                          "how": "CUDA events around one call that follows an unrelated elementwise kernel, cold W_trim copy"},
        "static_weights": {"us_per_call": round(us_static / world, 3),
                           "how": "same region with VT_HEAD_STATIC_WEIGHTS (W_trim declared constant: weight tiles are "
                                  "requested ahead of the stream-order wait)"},
        "clocks": clocks,
        "e2e": {"value": round(e2e_us / world, 3), "unit": UNIT, "h2d_bytes_per_step": M * d * 2,
                "d2h_bytes_per_step": M * k * 8, "steps": e2e_steps},
        "gpu_launches": args.steps * launches_per_call,
        "once_per_model": once,
    }

    if rank == 0 and world == 1:
        if not args.no_curve:
            line["curve"] = latency_curve(vt, torch, W_full, ranking, case, l2, peak_gbs, not args.no_graph)
            del W_full
            torch.cuda.empty_cache()
            line["fixed_vs_head"] = fixed_vs_head(vt, torch, line["curve"], d, V, l2, peak_gbs)
            line["other_workloads"] = config_timings(vt, torch, l2, peak_gbs, not args.no_graph)
        line["cpu_baseline"] = cpu_baseline(case)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_profile(args):
    """A few launches of one kernel family on a small device footprint, for ncu (never a benchmark number)."""
    import torch

    import paper_2603_05210_b200 as vt
    torch.cuda.set_device(0)
    vt.lib()
    gen = torch.Generator(device="cuda").manual_seed(3)
    V = inputs.V_LLAMA3
    if args.profile == "head":
        d, Vt, M, k = args.d, args.vtrim, args.m or 8, args.k
        nc = max(2, min(8, -(-400_000_000 // (Vt * d * 2))))            # copies beyond L2 in total, a few hundred MB
        copies = [(torch.randn((Vt, d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16) for _ in range(nc)]
        h = torch.randn((M, d), device="cuda", generator=gen).to(torch.bfloat16)
        d2t = torch.arange(Vt, dtype=torch.int32, device="cuda")
        ws = vt.new_workspace(vt.vt_workspace_bytes(M, k))
        for i in range(args.warmup + args.steps):
            vt.vt_draft_head(h, copies[i % nc], d2t, k, workspace=ws)
        assert vt.vt_last_status(ws) == vt.VT_OK
        print(json.dumps({"profile": "head", "d": d, "V_trim": Vt, "M": M, "k": k, "calls": args.warmup + args.steps,
                          "launches_per_call": vt.vt_last_launch_count()}))
        return
    d = args.d
    W_full = (torch.randn((V, d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16)
    tokens = inputs.zipf_token_stream(V, 1.05, 10_000_000, 5000)
    order, _ = inputs.frequency_ranking(tokens, V)
    keep = to_dev(np.ascontiguousarray(order[:args.vtrim]), torch)
    tok = [to_dev(tokens, torch) for _ in range(4)]                     # 160 MB of ids: beyond L2
    cov_ws = torch.empty(vt.vt_coverage_workspace_bytes(V), dtype=torch.uint8, device="cuda")
    W_trim = vt.vt_compact_head(W_full, keep)
    for i in range(max(1, args.steps)):
        vt.vt_compact_head(W_full, keep, out=W_trim)
        vt.vt_coverage_enqueue(tok[i % 4], keep, V, cov_ws)
    covered, frac = vt.vt_coverage_result(cov_ws, tokens.size)
    h3 = torch.randn((8, 3 * d), device="cuda", generator=gen).to(torch.bfloat16)
    Wf = (torch.randn((d, 3 * d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16)
    vt.vt_fuse_features(h3, Wf)
    sel = vt.vt_select_vocab(tok[0], V, d, 2.0 * 3 * d * d + 486.5e6, 0.5, 0.9, 1000, 64000)
    torch.cuda.synchronize()
    print(json.dumps({"profile": "aux", "coverage": frac, "k_star": sel["k_star"]}))


def bench_config(workload, cold, step, launch, parallelism, calls_per_s):
    """Both arms print the same keys, so that their configurations can be compared field by field."""
    return {"workload": workload, "cold": cold, "step": step, "launch": launch, "parallelism": parallelism,
            "calls_per_s": calls_per_s}


def event_us(torch, fn, reps):
    """Median CUDA-event time of fn() in us, one event pair per call, after one untimed call."""
    fn()
    pairs = []
    torch.cuda.synchronize()
    hold_gpu(torch)
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    return float(np.median([a.elapsed_time(b) for a, b in pairs])) * 1000.0


def once_per_model(vt, torch, W_full, keep, W_trim, tok_dev, tokens, d, V, peak_gbs):
    """The steps that run once per model: head compaction (row gather: read + write of the kept rows) at the bench
    size and at the untrimmed size, the coverage count (Eq. 2: one read of the token stream) on the 1M- and a
    10M-token stream, and the paper's selection step.  Device-timed; each with its own roofline fraction."""
    out = {}
    Vt = keep.numel()
    us = event_us(torch, lambda: vt.vt_compact_head(W_full, keep, out=W_trim), 10)
    gbs = 4 * d * Vt / us / 1e3
    out["compact"] = [{"V_trim": Vt, "d": d, "us": round(us, 2), "GBs": round(gbs, 1), "frac": round(gbs / peak_gbs, 4),
                       "bytes": 4 * d * Vt, "bound": "hbm read + write"}]
    ident = torch.arange(V, dtype=torch.int32, device="cuda")
    big = torch.empty_like(W_full)
    us = event_us(torch, lambda: vt.vt_compact_head(W_full, ident, out=big), 5)
    gbs = 4 * d * V / us / 1e3
    out["compact"].append({"V_trim": V, "d": d, "us": round(us, 2), "GBs": round(gbs, 1), "frac": round(gbs / peak_gbs, 4),
                           "bytes": 4 * d * V, "bound": "hbm read + write"})
    del big
    torch.cuda.empty_cache()
    cov_ws = torch.empty(vt.vt_coverage_workspace_bytes(V), dtype=torch.uint8, device="cuda")
    covered, frac = vt.vt_coverage(tok_dev, keep, V, cov_ws)
    out["coverage_value"] = frac
    out["coverage"] = []
    tok10 = torch.from_numpy(inputs.zipf_token_stream(V, 1.05, 10_000_000, 5000)).cuda()
    for t in (tok_dev, tok10):
        n = t.numel()
        us = event_us(torch, lambda: vt.vt_coverage_enqueue(t, keep, V, cov_ws), 20)
        gbs = 4 * n / us / 1e3
        out["coverage"].append({"tokens": n, "us": round(us, 2), "GBs": round(gbs, 1), "frac": round(gbs / peak_gbs, 4),
                                "bytes": 4 * n, "what": "counter clear + one kernel (bitmap built per CTA in shared memory, then the count), no host read"})
    t0 = time.perf_counter()
    for _ in range(10):
        vt.vt_coverage(tok_dev, keep, V, cov_ws)
    out["coverage_us_incl_sync"] = round((time.perf_counter() - t0) * 1e5, 2)
    del tok10
    # the paper's selection step (Eq. 1-5 as an exhaustive scan) on the same stream, Table 1 constants
    F_fixed = 2.0 * (3 * d) * d + 436.2e6 + 50.3e6
    sel_ws = torch.empty(vt.vt_select_workspace_bytes(V), dtype=torch.uint8, device="cuda")
    sel = vt.vt_select_vocab(tok_dev, V, d, F_fixed, 0.5, 0.9, 1000, 64000, workspace=sel_ws)
    t0 = time.perf_counter()
    for _ in range(5):
        sel = vt.vt_select_vocab(tok_dev, V, d, F_fixed, 0.5, 0.9, 1000, 64000, workspace=sel_ws)
    out["select_vocab_us_incl_sync"] = round((time.perf_counter() - t0) * 2e5, 1)
    out["select_vocab"] = {"alpha": 0.5, "c_min": 0.9, "k_range": [1000, 64000], "k_star": sel["k_star"],
                           "C": round(sel["C"], 6), "R": round(sel["R"], 6), "U": round(sel["U"], 6),
                           "unique_coverage": round(sel["unique"], 6)}
    return out


def latency_curve(vt, torch, W_full, ranking, case, l2, peak_gbs, use_graph=True):
    """us/call and roofline fraction over V_trim x M at d=4096 (the measured latency-vs-vocabulary curve): back-to-back
    calls (graph replay) and, beside them, single calls behind an unrelated kernel."""
    d, k = case.d, 8
    order = ranking[0]
    out = []
    for Vt in CURVE_VT:
        keep = to_dev(np.ascontiguousarray(order[:Vt]), torch)
        W_trim = vt.vt_compact_head(W_full, keep)
        free, _ = torch.cuda.mem_get_info()
        nc = n_copies_for_cold(W_trim.numel() * 2, l2, free)
        copies = [W_trim] + [W_trim.clone() for _ in range(nc - 1)]
        for M in CURVE_M:
            h = to_dev(inputs.hidden_states_bf16(M, d, 77 + M).view(np.int16), torch, torch.bfloat16)
            kk = min(k, Vt)
            steps = 480 if Vt <= 32000 else 120
            ms, _ = time_head(vt, torch, h, copies, keep, kk, steps, 20, use_graph=use_graph)
            us = ms * 1000.0 / steps
            us_iso = float(np.median(time_isolated(vt, torch, h, copies, keep, kk, n_calls=60)))
            by = head_bytes(d, Vt, M, kk)
            gbs = by / (us * 1e-6) / 1e9
            out.append({"V_trim": Vt, "M": M, "us_per_call": round(us, 2), "GBs": round(gbs, 1),
                        "frac": round(gbs / peak_gbs, 4), "us_isolated": round(us_iso, 2),
                        "frac_isolated": round(by / (us_iso * 1e-6) / 1e9 / peak_gbs, 4)})
        del copies, W_trim
        torch.cuda.empty_cache()
    return out


def fixed_vs_head(vt, torch, curve, d, V, l2, peak_gbs, M=8):
    """The paper's cost model (Section 2.3, Table 1, Eq. 3) beside what the same split costs on this GPU.

    Eq. 3 predicts the latency reduction of a draft vocabulary of size k from FLOPs: R(k) = 1 - (F_fixed + 2dk) /
    (F_fixed + 2dV), with F_fixed = fusion + attention + feed-forward (Table 1; the last two are taken as printed).
    Measured here: the feature-fusion projection (3d -> d, the one fixed component this library runs) and the head at
    every V_trim of the curve, M draft rows.  R_head_measured(k) = 1 - t_head(k) / t_head(V) is the measured counterpart
    of Eq. 3 for the head alone (F_fixed = 0); with the measured fusion time added on both sides it is
    R_fuse_head_measured(k).  On a bandwidth-bound GPU a fixed cost per call flattens both against the FLOPs proxy."""
    gen = torch.Generator(device="cuda").manual_seed(11)
    nc = n_copies_for_cold(d * 3 * d * 2, l2, torch.cuda.mem_get_info()[0])
    Wf = [(torch.randn((d, 3 * d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16) for _ in range(nc)]
    h3 = torch.randn((M, 3 * d), device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty((M, d), dtype=torch.bfloat16, device="cuda")
    ws = vt.new_workspace(vt.vt_workspace_bytes(M, 1))
    i = [0]

    def call():
        vt.vt_fuse_features(h3, Wf[i[0] % nc], out=out, workspace=ws)
        i[0] += 1

    for _ in range(10):
        call()
    steps = 240
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    hold_gpu(torch)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    assert vt.vt_last_status(ws) == vt.VT_OK
    t_fuse = e0.elapsed_time(e1) * 1000.0 / steps
    fuse_bytes = 2 * d * 3 * d + 2 * M * 3 * d + 2 * M * d
    F_fixed = 2.0 * (3 * d) * d + 436.2e6 + 50.3e6
    heads = {r["V_trim"]: r["us_per_call"] for r in curve if r["M"] == M}
    t_full = heads.get(V)
    rows = []
    for Vt in sorted(heads):
        r_eq3 = 1.0 - (F_fixed + 2.0 * d * Vt) / (F_fixed + 2.0 * d * V)
        row = {"V_trim": Vt, "t_head_us": heads[Vt], "R_eq3": round(r_eq3, 4),
               "R_eq3_head_only": round(1.0 - Vt / V, 4)}
        if t_full:
            row["R_head_measured"] = round(1.0 - heads[Vt] / t_full, 4)
            row["R_fuse_head_measured"] = round(1.0 - (t_fuse + heads[Vt]) / (t_fuse + t_full), 4)
        rows.append(row)
    return {"M": M, "d": d, "t_fuse_us": round(t_fuse, 2), "fuse_bytes": fuse_bytes,
            "fuse_GBs": round(fuse_bytes / t_fuse / 1e3, 1), "fuse_frac": round(fuse_bytes / t_fuse / 1e3 / peak_gbs, 4),
            "launch": "eager calls through the binding, back to back, cold copies of W_fuse",
            "table1_flops": {"fusion": 2.0 * 3 * d * d, "attention": 436.2e6, "feed_forward": 50.3e6, "head_full": 2.0 * d * V},
            "rows": rows}


def config_timings(vt, torch, l2, peak_gbs, use_graph=True):
    """us/call of the other benchmark workloads (shapes of the five configurations; random device-side weights,
    since only the shapes matter for the time).  The 95 % prefix of the fifth follows the input recipe."""
    V = inputs.V_LLAMA3
    tokens = inputs.zipf_token_stream(V, 1.05, 10_000_000, 5000)
    _, sorted_counts = inputs.frequency_ranking(tokens, V)
    vt95 = int(inputs.smallest_prefix_with_coverage(sorted_counts, 19, 20))
    shapes = [("cfg1", 2048, 4096, 1, 1)]
    shapes += [("cfg2", 3072, v, 1, 1) for v in (4096, 8192, 16384, 32000, V)]
    shapes += [("cfg4", 4096, 16384, m, 10) for m in (16, 64, 256)]
    shapes += [("cfg5 trimmed to 95 % coverage", 5120, vt95, 32, 8), ("cfg5 untrimmed", 5120, V, 32, 8)]
    out = []
    gen = torch.Generator(device="cuda").manual_seed(7)
    for name, d, Vt, M, k in shapes:
        free, _ = torch.cuda.mem_get_info()
        nc = n_copies_for_cold(Vt * d * 2, l2, free)
        copies = [(torch.randn((Vt, d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16) for _ in range(nc)]
        h = torch.randn((M, d), device="cuda", generator=gen).to(torch.bfloat16)
        d2t = torch.arange(Vt, dtype=torch.int32, device="cuda")
        steps = 480 if Vt * d <= 32000 * 4096 else 120
        ms, launches = time_head(vt, torch, h, copies, d2t, k, steps, 20, use_graph=use_graph)
        us = ms * 1000.0 / steps
        us_iso = float(np.median(time_isolated(vt, torch, h, copies, d2t, k, n_calls=60)))
        by = head_bytes(d, Vt, M, k)
        gbs = by / (us * 1e-6) / 1e9
        row = {"config": name, "d": d, "V_trim": Vt, "M": M, "k": k, "us_per_call": round(us, 2),
               "GBs": round(gbs, 1), "frac": round(gbs / peak_gbs, 4), "us_isolated": round(us_iso, 2),
               "frac_isolated": round(by / (us_iso * 1e-6) / 1e9 / peak_gbs, 4), "launches_per_call": launches}
        if M >= 128:      # where the tensor pipe is co-limiting: the contraction's share of the dense bf16 peak
            row["TFLOPs"] = round(2.0 * M * d * Vt / (us * 1e-6) / 1e12, 1)
        out.append(row)
        del copies
        torch.cuda.empty_cache()
    return out


ONE_THREAD_SNIPPET = """
import sys, time, numpy as np
sys.path.insert(0, {root!r})
import oracle
from paper_2603_05210_b200 import inputs
rows, d, M, k, seed = {rows}, {d}, {M}, {k}, {seed}
W = inputs.normal_bf16((rows, d), 0.02, seed)
h = inputs.hidden_states_bf16(M, d, seed, row_scale=(0.5, 2.0))
d2t = np.arange(rows, dtype=np.int32)
best = 1e30
for _ in range(2):
    t0 = time.perf_counter(); oracle.draft_head(h, W, d2t, k); best = min(best, time.perf_counter() - t0)
print(oracle.num_threads(), best)
"""


def cpu_baseline(case):
    """The oracle as it stands, timed on this host on the bench workload: one full call on all cores (best of 3),
    and on one thread on a sample of the vocabulary rows scaled to the full call."""
    import oracle
    W_trim = oracle.compact(case.W_full, case.keep_ids)
    best = float("inf")
    for _ in range(3):
        t0 = time.perf_counter()
        oracle.draft_head(case.h, W_trim, case.d2t, case.k)
        best = min(best, time.perf_counter() - t0)
    out = {"value": round(best * 1e6, 1), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "the whole bench workload, one full call, best of 3"}
    rows = 2000
    try:
        env = dict(os.environ, OMP_NUM_THREADS="1")
        r = subprocess.run([sys.executable, "-c", ONE_THREAD_SNIPPET.format(root=ROOT, rows=rows, d=case.d, M=case.M, k=case.k,
                                                                           seed=WORKLOAD["seed"])],
                           capture_output=True, text=True, env=env, timeout=300)
        nthreads, t = r.stdout.split()[-2:]
        out["one_thread"] = {"value": round(float(t) * 1e6 * case.V_trim / rows, 1), "unit": UNIT, "cores": int(nthreads),
                             "sample": f"the first {rows} of {case.V_trim} vocabulary rows (all {case.M} draft rows), "
                                       f"scaled by {case.V_trim}/{rows}, best of 2"}
    except Exception as ex:       # the one-thread figure is an extra; the all-cores figure above is the baseline
        out["one_thread"] = {"value": None, "why": str(ex)[:200]}
    return out


def run_reference(args):
    """The reference arm: the CPU oracle on the same workload and metric (a deliberately plain program)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = WORKLOAD
    d, V, Vt, M, k = w["d"], w["V_full"], w["V_trim"], w["M"], w["k"]
    tokens = inputs.zipf_token_stream(V, 1.1, 1_000_000, w["seed"])
    ranking = inputs.frequency_ranking(tokens, V)
    # weights only for the sampled rows: the oracle's cost per row does not depend on their values' origin
    rng_rows = 2048
    case = inputs.make_case("ref", d, rng_rows, M, k, w["seed"], V_full=V, ranking=ranking,
                            W_full=inputs.normal_bf16((rng_rows, d), 0.02, w["seed"]),
                            row_scale=(0.5, 2.0))
    W = case.W_full
    d2t = np.ascontiguousarray(ranking[0][:rng_rows])
    t0 = time.perf_counter()
    oracle.draft_head(case.h, W, d2t, k)
    probe = time.perf_counter() - t0
    per_row = probe / rng_rows
    total_steps = args.steps + args.warmup
    rows = int(max(256, min(Vt, 120.0 / max(total_steps, 1) / per_row)))
    if rows > rng_rows:
        W = inputs.normal_bf16((rows, d), 0.02, w["seed"])
        d2t = np.ascontiguousarray(ranking[0][:rows])
    else:
        W, d2t = W[:rows], d2t[:rows]
    for _ in range(args.warmup):
        oracle.draft_head(case.h, W, d2t, min(k, rows))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.draft_head(case.h, W, d2t, min(k, rows))
    dt = (time.perf_counter() - t0) / args.steps
    us_full = dt * 1e6 * Vt / rows
    line = {"impl": "reference", "metric": METRIC, "value": round(us_full, 1), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 4),
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": bench_config(WORKLOAD_NAME, cold="host memory (the oracle reads its inputs from RAM)",
                                   step="one oracle.draft_head call on a sample of the vocabulary rows, scaled",
                                   launch="host function call", parallelism="host threads",
                                   calls_per_s=round(1e6 / us_full, 3)),
            "cpu_baseline": {"value": round(us_full, 1), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"each step runs the oracle on the first {rows} of {Vt} vocabulary rows "
                                       f"(all {M} draft rows); value scaled by {Vt}/{rows}"},
            "e2e": {"value": round(us_full, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-curve", action="store_true")
    ap.add_argument("--m", type=int, default=None, help="draft rows M instead of the workload's 8 (not the headline)")
    ap.add_argument("--no-graph", action="store_true", help="launch every timed call through the binding instead of a CUDA graph")
    ap.add_argument("--profile", default=None, choices=["head", "aux"],
                    help="a short run for a profiler instead of the benchmark: 'head' = warm-up + --steps eager head calls on "
                         "--d/--vtrim/--m/--k (random weights, cold copies); 'aux' = compaction, coverage, selection, fusion once each")
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--vtrim", type=int, default=32000)
    ap.add_argument("--k", type=int, default=8)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.profile:
        run_profile(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
