"""Benchmark of the TurboQuant hot path on B200.

One "step" = one pass of the whole hot path over one batch of synthetic vectors:
  Quant_prod (rotate, nearest centroid, pack, residual, QJL signs, norms) of n vectors, then the
  packed-code inner-product scan of nq rotated queries against those codes with top-k selection.
Workload at N = 1: d = 1536, b = 4 (3-bit MSE stage + 1-bit QJL), n = 1,000,000 embedding-like
vectors, nq = 8 queries, k = 100 (the configuration the headline metric is quoted on).

  python bench.py --gpus N --steps K --warmup W          (N > 1: launched by torch.distributed.run)
  python bench.py --impl reference ...                   (times the CPU oracle on a bounded sample)

Prints ONE JSON line.  `value` is vectors/s through the whole step with inputs resident in HBM;
`e2e` is the same with the inputs starting in pinned host memory and the codes and top-k
returned to the host.  Vectors shard across GPUs with no exchange in the quantise phase; the
top-k lists of the shards are all-gathered (nq*k*8 bytes per rank) and merged.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "quantize+scan throughput at d=1536, b=4 (TurboQuant_prod), n=1M, nq=8, top-100"
UNIT = "vectors/s"
WORKLOAD = {"name": "c4", "bits": 4, "mode": "prod", "n": 1_000_000, "nq": 8, "k": 100}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--n", type=int, default=WORKLOAD["n"], help="vectors per GPU (smaller only for profiling runs)")
    ap.add_argument("--nq", type=int, default=WORKLOAD["nq"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv", action="store_true", help="run the KV-cache decode leg even when --n is reduced (profiling runs)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples (one every 25 ms) from start() to stop(), each with the
    time it was taken, so that every timed leg can report the SM clock it ran at."""
    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.samples = []      # (epoch seconds, sm MHz, max MHz, set of active reasons)

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "25", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        self.proc = None
        import datetime
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 10:
                continue
            try:
                t = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                sm, mx = float(f[2]), float(f[3])
            except ValueError:
                continue
            self.samples.append((t, sm, mx, {n for n, v in zip(self.NAMES, f[6:10]) if v.lower().startswith("active")}))

    def window(self, t0: float, t1: float):
        """Median SM clock and the throttle reasons seen between two time.time() stamps (the nearest sample
        when the window is shorter than the sampling period)."""
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"], "samples": 0}
        inside = [x for x in self.samples if t0 <= x[0] <= t1]
        if not inside:
            mid = 0.5 * (t0 + t1)
            inside = [min(self.samples, key=lambda x: abs(x[0] - mid))]
        sm = [x[1] for x in inside]
        busy = [v for v in sm if v > 0.5 * max(sm)] or sm
        reasons = set().union(*[x[3] for x in inside])
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(x[2] for x in inside), "reasons": sorted(reasons),
                "samples": len(inside)}


# ------------------------------------------------------------------------------------------
def cpu_oracle_sample(d, bits, nq, k, sample_n, Pi=None, S=None):
    """Times the oracle (as it stands) on `sample_n` vectors of the workload: Quant_prod, then
    DeQuant_prod + inner products + top-k for nq queries.  Returns (seconds, threads)."""
    import numpy as np
    import threadpoolctl

    import tq_workloads as wl
    from oracle import turboquant_oracle as orc
    cfg = wl.CONFIGS[WORKLOAD["name"]]
    X = wl.database(cfg, sample_n).numpy()
    Q = wl.queries(cfg, nq).numpy()
    Pi = orc.rotation(d, cfg.pi_seed).astype(np.float32) if Pi is None else Pi
    S = orc.projection(d, cfg.s_seed).astype(np.float32) if S is None else S
    c = orc.codebook(d, bits - 1).astype(np.float32)
    threads = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info() if p.get("user_api") == "blas"] or [1])
    t0 = time.perf_counter()
    idx, z, gamma, nu = orc.quant_prod(X, Pi, S, c)
    Xh = orc.dequant_prod(idx, z, gamma, nu, Pi, S, c)
    orc.topk(orc.score(Q, Xh), min(k, sample_n))
    return time.perf_counter() - t0, threads, (Pi, S)


def run_reference(args):
    """The reference arm is the CPU oracle: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import tq_workloads as wl
    d = wl.CONFIGS[WORKLOAD["name"]].d
    sample = 8192
    mats = None
    times = []
    for it in range(args.warmup + args.steps):
        dt, threads, mats = cpu_oracle_sample(d, WORKLOAD["bits"], args.nq, WORKLOAD["k"], sample, *(mats or (None, None)))
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = sample * len(times) / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"c4 d={d} prod b=4, sample of {sample} vectors per step, nq={args.nq}, k=100"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{sample} vectors x {args.nq} queries per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
def run_b200(args):
    import numpy as np  # noqa: F401
    import torch
    import torch.distributed as dist

    import paper_2504_19874_b200 as tq
    import tq_workloads as wl
    from paper_2504_19874_b200 import build as tq_build
    from paper_2504_19874_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    tq_build.build()
    tq.lib()
    peaks = measured_peaks()
    full = args.n == WORKLOAD["n"] and world == 1     # the stand-alone legs of the other configurations run at full size only

    cfg = wl.CONFIGS[WORKLOAD["name"]]
    d, bits, n, nq, k = cfg.d, WORKLOAD["bits"], args.n, args.nq, WORKLOAD["k"]
    Pi = tq.tq_rotation(d, cfg.pi_seed)
    S = tq.tq_rotation(d, cfg.s_seed, tq.TQ_GAUSSIAN)
    cent, _ = tq.tq_codebook(d, bits - 1)
    plan = tq.Plan(d, bits, tq.TQ_PROD, Pi, S, cent)
    plan.set_layout(tq.TQ_LAYOUT_NIBBLE)               # the code layout of the table-lookup scan (same bytes per vector)

    # Synthetic inputs, resident in HBM before the timed region (each rank draws its own shard).
    X = wl.make_vectors(cfg, n, cfg.data_seed + 1000 * rank, dev)
    Q = wl.queries(cfg, nq, dev)
    idx = torch.empty((n, plan.idx_row_bytes), dtype=torch.uint8, device=dev)
    qjl = torch.empty((n, plan.qjl_row_bytes), dtype=torch.uint8, device=dev)
    gamma = torch.empty(n, dtype=torch.float32, device=dev)
    norms = torch.empty(n, dtype=torch.float32, device=dev)
    scratch_bytes = max(tq.tq_workspace_bytes(plan, tq.TQ_OP_QUANTIZE, n), 16)
    scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=dev)
    ws = torch.empty(max(tq.tq_workspace_bytes(plan, tq.TQ_OP_TOPK, n, nq, k), 16), dtype=torch.uint8, device=dev)
    top_s = torch.empty((nq, k), dtype=torch.float32, device=dev)
    top_i = torch.empty((nq, k), dtype=torch.int32, device=dev)
    merged_s = torch.empty((nq, k), dtype=torch.float32, device=dev)
    merged_i = torch.empty((nq, k), dtype=torch.int32, device=dev)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    phase_ms = {"quantize": [], "scan": []}

    def step(record: bool):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        tq.tq_quantize_prod(plan, X, idx, qjl, gamma, norms, scratch)
        e1.record()
        tq.tq_topk(plan, Q, n, idx, qjl, gamma, norms, k, top_s, top_i, ws)
        if world > 1:   # local best lists -> all ranks -> global best list (ids made global by the shard offset)
            cand_s, cand_i = sharding.gather_candidates(top_s, top_i, rank * n)
            tq.tq_select_topk(cand_s, cand_i, k, merged_s, merged_i)
        e2.record()
        if record:
            return e0, e1, e2
        return None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # The clock sampler runs from before the warm-up steps to the end of the last stand-alone leg; every leg
    # reports the median SM clock of the samples taken while it ran.
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step(False)
    barrier()
    launches0 = tq.tq_launch_count()
    barrier()
    t_start = ev()
    t_end = ev()
    wall0 = time.time()
    t_start.record()
    evs = [step(True) for _ in range(args.steps)]
    t_end.record()
    barrier()
    wall1 = time.time()
    launches = tq.tq_launch_count() - launches0
    total_ms = t_start.elapsed_time(t_end)
    for e0, e1, e2 in evs:
        phase_ms["quantize"].append(e0.elapsed_time(e1))
        phase_ms["scan"].append(e1.elapsed_time(e2))
    if world > 1:
        t = torch.tensor([total_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = t.item()
    ms_per_step = total_ms / args.steps
    value = world * n / (ms_per_step * 1e-3)
    leg_windows = {"steps": (wall0, wall1)}

    def time_call(fn, name=None, min_ms=150.0, max_reps=400):
        """Mean CUDA-event time of fn over enough repetitions to last min_ms (so that the clock sampler sees the
        leg); the leg's wall-clock window is kept under `name`."""
        for _ in range(2):
            fn()
        a0, a1 = ev(), ev()
        barrier()
        a0.record()
        fn()
        a1.record()
        barrier()
        reps = int(min(max_reps, max(3, math.ceil(min_ms / max(a0.elapsed_time(a1), 1e-3)))))
        w0 = time.time()
        a0.record()
        for _ in range(reps):
            fn()
        a1.record()
        barrier()
        if name:
            leg_windows[name] = (w0, time.time())
        return a0.elapsed_time(a1) / reps

    def cool():
        # the scans are issue-bound: half a second lets the SM clock recover from the power-capped GEMMs before
        # a scan is timed alone (each leg reports the clock it saw)
        torch.cuda.synchronize()
        time.sleep(0.5)

    def scan_legs(pl, label, nn, codes, Qall, kk, few=(1, 2, 8), many=None, bytes_per_vec=None):
        """Stand-alone timings of the scan on resident codes: whole tq_score calls, the scan alone on prepared
        queries, top-k; optionally a many-query top-k (queries/s and the fraction of the tensor bound)."""
        ci, cq, cg, cnm = codes
        cb = nn * bytes_per_vec
        out = []
        cool()
        for rq in few:
            Qr = Qall[:rq].contiguous()
            w = torch.empty(max(tq.tq_workspace_bytes(pl, tq.TQ_OP_TOPK, nn, rq, kk), 16), dtype=torch.uint8, device=dev)
            sc = torch.empty((rq, nn), dtype=torch.float32, device=dev)
            ts_, ti_ = torch.empty((rq, kk), dtype=torch.float32, device=dev), torch.empty((rq, kk), dtype=torch.int32, device=dev)
            prep = torch.empty(max(tq.tq_query_bytes(pl, rq), 256), dtype=torch.uint8, device=dev)
            tq.tq_query_prepare(pl, Qr, prep)
            ms_call = time_call(lambda: tq.tq_score(pl, Qr, nn, ci, cq, cg, cnm, sc, w), f"{label}:score{rq}")
            ms_scan = time_call(lambda: tq.tq_score_prepared(pl, prep, rq, nn, ci, cq, cg, cnm, sc), f"{label}:scan{rq}")
            ms_topk = time_call(lambda: tq.tq_topk(pl, Qr, nn, ci, cq, cg, cnm, kk, ts_, ti_, w), f"{label}:topk{rq}")
            gbs = lambda ms: cb / (ms * 1e-3) / 1e9
            out.append({"nq": rq, "score_call_ms": ms_call, "scan_prepared_ms": ms_scan, "topk_ms": ms_topk,
                        "score_call_codes_gbs": gbs(ms_call), "scan_prepared_codes_gbs": gbs(ms_scan),
                        "score_call_frac_hbm": gbs(ms_call) / peaks["hbm_gbs"], "scan_prepared_frac_hbm": gbs(ms_scan) / peaks["hbm_gbs"],
                        "scan_prepared_frac_nominal_8tbs": gbs(ms_scan) / 8000.0, "legs": [f"{label}:score{rq}", f"{label}:scan{rq}", f"{label}:topk{rq}"]})
            del w, sc, prep
        res = {"few_queries": out}
        if many:
            Qm = Qall[:many].contiguous()
            w = torch.empty(max(tq.tq_workspace_bytes(pl, tq.TQ_OP_TOPK, nn, many, kk), 16), dtype=torch.uint8, device=dev)
            ts_, ti_ = torch.empty((many, kk), dtype=torch.float32, device=dev), torch.empty((many, kk), dtype=torch.int32, device=dev)
            ms_m = time_call(lambda: tq.tq_topk(pl, Qm, nn, ci, cq, cg, cnm, kk, ts_, ti_, w), f"{label}:topk{many}", min_ms=0.0, max_reps=2)
            # dense-contraction view of the many-query regime: 2 d MACs per (query, vector) for the centroid term and
            # the sign term each (one for TQ_MSE), against the measured bf16 rate
            terms = 2 if pl.mode == tq.TQ_PROD else 1
            tf = 2.0 * terms * many * nn * pl.d / (ms_m * 1e-3) / 1e12
            res["many_queries"] = {"nq": many, "top_k": kk, "topk_ms": ms_m, "queries_per_s": many / (ms_m * 1e-3),
                                   "algorithmic_tflops": tf, "frac_bf16_sustained": tf / peaks["bf16_tflops_sustained"],
                                   "leg": f"{label}:topk{many}"}
            del w
        return res

    code_bytes_vec = plan.idx_row_bytes + plan.qjl_row_bytes + 8
    code_bytes = n * code_bytes_vec
    many_q = 10_000 if full else 256
    Qbig = wl.make_vectors(cfg, max(many_q, 8), cfg.query_seed + 7, dev) if world == 1 else Q
    main_scan = scan_legs(plan, "c4b4", n, (idx, qjl, gamma, norms), Qbig if world == 1 else Q, k,
                          few=(1, 2, 8) if nq >= 8 else (1, 2), many=many_q if world == 1 else None, bytes_per_vec=code_bytes_vec)
    # the allocation-free entry point (library-owned scratch), same kernels
    static_leg = []
    sc_st = torch.empty((8, n), dtype=torch.float32, device=dev)
    for rq in (1, 8):
        Qr = Qbig[:rq].contiguous()
        ms_st = time_call(lambda: tq.tq_score_static(plan, Qr, n, idx, qjl, gamma, norms, sc_st[:rq]), f"c4b4:static{rq}")
        static_leg.append({"nq": rq, "score_static_ms": ms_st, "codes_gbs": code_bytes / (ms_st * 1e-3) / 1e9})
    del sc_st

    # ---- the same workload at TurboQuant_mse b = 2 (the metric is quoted at b = 2 and b = 4) ----
    cent2, _ = tq.tq_codebook(d, 2)
    plan2 = tq.Plan(d, 2, tq.TQ_MSE, Pi, None, cent2)
    idx2 = torch.empty((n, plan2.idx_row_bytes), dtype=torch.uint8, device=dev)
    norms2 = torch.empty(n, dtype=torch.float32, device=dev)
    scratch2 = torch.empty(max(tq.tq_workspace_bytes(plan2, tq.TQ_OP_QUANTIZE, n), 16), dtype=torch.uint8, device=dev)
    ms_q2 = time_call(lambda: tq.tq_quantize_mse(plan2, X, idx2, norms2, scratch2), "c4b2:quantize", min_ms=0.0, max_reps=3)
    mse_scan = scan_legs(plan2, "c4b2", n, (idx2, None, None, norms2), Qbig, k, few=(1, 8), many=many_q if full else None,
                         bytes_per_vec=plan2.idx_row_bytes + 4)
    mse_b2 = {"workload": f"c4: d={d}, TurboQuant_mse b=2, n={n}, top-{k}",
              "quantize_ms": ms_q2, "quantize_vectors_per_s": n / (ms_q2 * 1e-3),
              "quantize_frac_bf16_sustained": 2.0 * n * d * d / (ms_q2 * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
              "quantize_frac_of_three_pass_bound": 3 * 2.0 * n * d * d / (ms_q2 * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
              **mse_scan}
    del idx2, norms2, scratch2, plan2

    # ---- the other vector configurations at full size: quantise time and scan times (c2: d = 200, b = 3;
    #      c5: d = 3072, b = 2 and 4), each with its own inputs ----
    other = None
    if full:
        other = []
        for cname, cbits, ck in (("c2", 3, 100), ("c5", 2, 10), ("c5", 4, 100)):
            cc = wl.CONFIGS[cname]
            dd, nn = cc.d, cc.n
            cent_c, _ = tq.tq_codebook(dd, cbits - 1)
            plan_c = tq.Plan(dd, cbits, tq.TQ_PROD, tq.tq_rotation(dd, cc.pi_seed), tq.tq_rotation(dd, cc.s_seed, tq.TQ_GAUSSIAN), cent_c)
            nibble = cbits == 4
            if nibble:
                plan_c.set_layout(tq.TQ_LAYOUT_NIBBLE)
            Xc = wl.make_vectors(cc, nn, cc.data_seed, dev)
            Qc = wl.make_vectors(cc, 10_000, cc.query_seed + 7, dev)
            ci = torch.empty((nn, max(plan_c.idx_row_bytes, 1)), dtype=torch.uint8, device=dev)
            cq = torch.empty((nn, plan_c.qjl_row_bytes), dtype=torch.uint8, device=dev)
            cg = torch.empty(nn, dtype=torch.float32, device=dev)
            cn = torch.empty(nn, dtype=torch.float32, device=dev)
            cs = torch.empty(max(tq.tq_workspace_bytes(plan_c, tq.TQ_OP_QUANTIZE, nn), 16), dtype=torch.uint8, device=dev)
            ms_q = time_call(lambda: tq.tq_quantize_prod(plan_c, Xc, ci, cq, cg, cn, cs), f"{cname}b{cbits}:quantize", min_ms=0.0, max_reps=2)
            del Xc, cs
            bpv = plan_c.idx_row_bytes + plan_c.qjl_row_bytes + 8
            legs = scan_legs(plan_c, f"{cname}b{cbits}", nn, (ci, cq, cg, cn), Qc, ck, few=(1, 8), many=10_000, bytes_per_vec=bpv)
            other.append({"workload": f"{cname}: d={dd}, TurboQuant_prod b={cbits}, n={nn}, top-{ck}",
                          "layout": "nibble" if nibble else "canonical",
                          "quantize_ms": ms_q, "quantize_vectors_per_s": nn / (ms_q * 1e-3),
                          "quantize_frac_bf16_sustained": 4.0 * nn * dd * dd / (ms_q * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                          "quantize_frac_of_three_pass_bound": 3 * 4.0 * nn * dd * dd / (ms_q * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                          **legs})
            del ci, cq, cg, cn, plan_c, Qc
            torch.cuda.empty_cache()

    # ---- KV-cache decode (config c3): one layer = 8 KV heads x 32768 tokens, 2.5 bits per channel, 32 query heads;
    #      enough layer copies that the codes exceed L2; tq_attend_decode, one call per layer.  Also other context
    #      lengths (random codes of the same shape) and a 3.5-bit split (64 channels at 4 bits + 64 at 3 bits). ----
    kv = None
    if n == WORKLOAD["n"] or args.kv:
        kv = kv_decode_legs(tq, wl, dev, peaks, time_call)

    # ---- end to end: inputs start in pinned host memory, codes and top-k go back to the host ----
    e2e = None
    if not args.no_e2e:
        chunk = 65536
        hX = torch.empty((n, d), dtype=torch.float32).pin_memory()
        hX.copy_(X)
        h_idx = torch.empty((n, plan.idx_row_bytes), dtype=torch.uint8).pin_memory()
        h_qjl = torch.empty((n, plan.qjl_row_bytes), dtype=torch.uint8).pin_memory()
        h_gamma = torch.empty(n, dtype=torch.float32).pin_memory()
        h_norms = torch.empty(n, dtype=torch.float32).pin_memory()
        h_ts = torch.empty((nq, k), dtype=torch.float32).pin_memory()
        h_ti = torch.empty((nq, k), dtype=torch.int32).pin_memory()
        hQ = Q.cpu().pin_memory()
        copy_stream = torch.cuda.Stream(device=dev)
        out_stream = torch.cuda.Stream(device=dev)
        stage = [torch.empty((chunk, d), dtype=torch.float32, device=dev) for _ in range(2)]
        dQ = torch.empty_like(Q)

        def e2e_step():
            main = torch.cuda.current_stream()
            ready = [None, None]
            freed = [None, None]
            for ci_, r0 in enumerate(range(0, n, chunk)):
                rows = min(chunk, n - r0)
                b = ci_ & 1
                with torch.cuda.stream(copy_stream):
                    if freed[b] is not None:
                        copy_stream.wait_event(freed[b])
                    stage[b][:rows].copy_(hX[r0:r0 + rows], non_blocking=True)
                    ready[b] = torch.cuda.Event()
                    ready[b].record(copy_stream)
                main.wait_event(ready[b])
                tq.tq_quantize_prod(plan, stage[b][:rows], idx[r0:r0 + rows], qjl[r0:r0 + rows], gamma[r0:r0 + rows],
                                    norms[r0:r0 + rows], scratch)
                freed[b] = torch.cuda.Event()
                freed[b].record(main)
                with torch.cuda.stream(out_stream):
                    out_stream.wait_event(freed[b])
                    h_idx[r0:r0 + rows].copy_(idx[r0:r0 + rows], non_blocking=True)
                    h_qjl[r0:r0 + rows].copy_(qjl[r0:r0 + rows], non_blocking=True)
                    h_gamma[r0:r0 + rows].copy_(gamma[r0:r0 + rows], non_blocking=True)
                    h_norms[r0:r0 + rows].copy_(norms[r0:r0 + rows], non_blocking=True)
            dQ.copy_(hQ, non_blocking=True)
            tq.tq_topk(plan, dQ, n, idx, qjl, gamma, norms, k, top_s, top_i, ws)
            h_ts.copy_(top_s, non_blocking=True)
            h_ti.copy_(top_i, non_blocking=True)
            done = torch.cuda.Event()
            done.record(out_stream)
            main.wait_event(done)

        e2e_step()
        barrier()
        a, b_ = ev(), ev()
        w0 = time.time()
        a.record()
        reps = max(1, min(args.steps, 3))
        for _ in range(reps):
            e2e_step()
        b_.record()
        barrier()
        leg_windows["e2e"] = (w0, time.time())
        e2e_ms = a.elapsed_time(b_) / reps
        if world > 1:
            t = torch.tensor([e2e_ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = t.item()
        h2d = n * d * 4 + nq * d * 4
        d2h = n * (plan.idx_row_bytes + plan.qjl_row_bytes + 8) + nq * k * 8
        e2e = {"value": world * n / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        del hX, stage

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    sampler.stop()
    clocks = sampler.window(*leg_windows["steps"])
    leg_clocks = {name: sampler.window(*w)["sm_mhz"] for name, w in leg_windows.items()}
    reasons_all = sorted(set().union(*[set(sampler.window(*w)["reasons"]) for w in leg_windows.values()]))

    q_ms = statistics.mean(phase_ms["quantize"])
    s_ms = statistics.mean(phase_ms["scan"])
    # Dominant kernels: the two d x d contractions of Quant_prod (4 n d^2 flops in all).
    gemm_flops = 4.0 * n * d * d
    achieved_tf = gemm_flops / (q_ms * 1e-3) / 1e12
    per_row = tq.tq_workspace_bytes(plan, tq.TQ_OP_QUANTIZE, 256) // 256      # scratch bytes per row of a launch
    rows_per_launch = min(n, scratch_bytes // max(per_row, 1) // 128 * 128)
    launches_per_step = math.ceil(n / max(rows_per_launch, 1))
    algo_bytes_row = 4 * d + plan.idx_row_bytes + plan.qjl_row_bytes + 8
    roofline = {"bound": "tensor", "kernel": f"tc::quantize_gemm_kernel on CTA pairs (Y = U Pi^T and Z = E S'^T, one launch of each per {rows_per_launch} rows)",
                "achieved": achieved_tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": achieved_tf / peaks["bf16_tflops_sustained"],
                "frac_of_three_pass_bound": 3.0 * achieved_tf / peaks["bf16_tflops_sustained"],
                "traffic": QUANTIZE_TRAFFIC_PER_98304_ROWS if d == 1536 else None,
                "traffic_source": "ncu capture of one rotate + one project launch of 98,304 rows (profile summary, not measured in this run) "
                                  "plus the bytes the split_rows launch of the block moves by definition",
                "algorithmic_bytes_per_launch": algo_bytes_row * rows_per_launch,
                "peak_source": f"bf16 sustained, of {peaks['source']}",
                "note": "achieved = algorithmic flops 4 n d^2 of the step / CUDA-event time of the quantise phase "
                        f"({launches_per_step} launches of each GEMM per step); fp32 fidelity is emulated with 3 bf16 MMA passes, "
                        "frac_of_three_pass_bound = 3 x frac is the fraction of that emulation's own tensor bound, frac is the headline"}
    few = {r["nq"]: r for r in main_scan["few_queries"]}
    best = few[1]
    roofline_scan = {"bound": "hbm", "kernel": "nscan::scan_nib_kernel (packed-code scan, one pass over the codes, nq <= 2, dense scores)",
                     "achieved": best["scan_prepared_codes_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": best["scan_prepared_frac_hbm"], "frac_of_nominal_8tbs": best["scan_prepared_frac_nominal_8tbs"],
                     "frac_whole_call": best["score_call_frac_hbm"],
                     "frac_nq8": few[8]["scan_prepared_frac_hbm"] if 8 in few else None,
                     "frac_nq8_whole_call": few[8]["score_call_frac_hbm"] if 8 in few else None,
                     "traffic": SCAN_TRAFFIC_PER_VECTOR * n,
                     "traffic_source": "ncu capture at n = 262,144 (205.9 MB read + 5.0 MB written), scaled by n",
                     "peak_source": f"copy bandwidth, of {peaks['source']}",
                     "note": "achieved = algorithmic code bytes (idx + qjl + gamma + nu = 776 B per vector) of one pass / "
                             "CUDA-event time of tq_score_prepared (the scan kernel alone; queries prepared once by "
                             "tq_query_prepare); frac_whole_call divides by the time of a whole tq_score call instead "
                             "(query rotation and operand set-up included)"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"c4: d={d}, TurboQuant_prod b={bits}, n={n} per GPU, nq={nq}, top-{k}",
                       "code_layout": "nibble (tq_plan_set_layout; same 776 bytes per vector as the bit streams)",
                       "l2": "inputs (6.1 GB of vectors, 0.78 GB of codes) are larger than L2; no flush needed"},
            "quantize_vectors_per_s": n / (q_ms * 1e-3), "quantize_ms": q_ms,
            "scan_ms": s_ms, "scan_queries_per_s": nq / (s_ms * 1e-3),
            "scan_codes_gbs": code_bytes / (s_ms * 1e-3) / 1e9, "scan_frac_hbm": code_bytes / (s_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "scan_regimes": main_scan["few_queries"], "scan_many_queries": main_scan.get("many_queries"),
            "score_static": static_leg, "mse_b2": mse_b2, "kv_decode": kv, "other_configs": other,
            "roofline": roofline, "roofline_scan": roofline_scan,
            "clocks": {**clocks, "reasons": reasons_all, "per_leg_sm_mhz": leg_clocks},
            "e2e": e2e, "gpu_launches": int(launches)}
    if not args.no_cpu_baseline:
        sample = 32768
        dt, threads, _ = cpu_oracle_sample(d, bits, nq, k, sample)
        line["cpu_baseline"] = {"value": sample / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{sample} vectors x {nq} queries, {dt:.1f} s"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes of the dominant kernels from ncu captures (one launch each; see the summaries under profiles/)
# rotate launch (680.8 MB read + 650.5 MB written) + project launch (690.2 + 71.4 MB) of the CTA-pair GEMM, from ncu;
# + the split_rows launch of the block (reads 98,304 x 6144 B, writes two bf16 limbs of the same size: 604 + 604 MB)
QUANTIZE_TRAFFIC_PER_98304_ROWS = (680.8e6 + 650.5e6) + (690.2e6 + 71.4e6) + 2 * 604.0e6
SCAN_TRAFFIC_PER_VECTOR = (205.9e6 + 5.0e6) / 262144


def kv_decode_legs(tq, wl, dev, peaks, time_call):
    import torch
    Kc, Vc, Qc = wl.kv_cache(device=dev)
    Hh, Tt, hd = Kc.shape
    grp = 64

    def kv_plan(b, mode, ps, ss):
        cent_g, _ = tq.tq_codebook(grp, b - 1 if mode == tq.TQ_PROD else b)
        return tq.Plan(grp, b, mode, tq.tq_rotation(grp, ps), tq.tq_rotation(grp, ss, tq.TQ_GAUSSIAN) if mode == tq.TQ_PROD else None, cent_g)

    def split(Xh):   # harness rule: the 64 channels of largest energy form the outlier group
        o = torch.topk(Xh.float().pow(2).sum(0), grp).indices.sort().values
        m = torch.ones(hd, dtype=torch.bool, device=dev)
        m[o] = False
        return o, torch.nonzero(m).flatten()

    chk = [split(Kc[h]) for h in range(Hh)]
    chv = [split(Vc[h]) for h in range(Hh)]
    code_keys = ("k_idx", "k_qjl", "k_gamma", "k_norms", "v_idx", "v_norms")

    def build_groups(kbits, vbits, tokens):
        pk = (kv_plan(kbits[0], tq.TQ_PROD, 72, 73), kv_plan(kbits[1], tq.TQ_PROD, 74, 75))
        pv = (kv_plan(vbits[0], tq.TQ_MSE, 76, 77), kv_plan(vbits[1], tq.TQ_MSE, 78, 79))
        groups = []
        for g in range(2):
            reps = (tokens + Tt - 1) // Tt          # longer contexts repeat the synthetic tokens
            Xk = torch.cat([Kc[h][:, chk[h][g]].repeat(reps, 1)[:tokens] for h in range(Hh)]).contiguous()
            Xv = torch.cat([Vc[h][:, chv[h][g]].repeat(reps, 1)[:tokens] for h in range(Hh)]).contiguous()
            rows = Xk.shape[0]
            gd = {"plan_k": pk[g], "plan_v": pv[g],
                  "k_idx": torch.empty((rows, pk[g].idx_row_bytes), dtype=torch.uint8, device=dev),
                  "k_qjl": torch.empty((rows, pk[g].qjl_row_bytes), dtype=torch.uint8, device=dev),
                  "k_gamma": torch.empty(rows, device=dev), "k_norms": torch.empty(rows, device=dev),
                  "v_idx": torch.empty((rows, pv[g].idx_row_bytes), dtype=torch.uint8, device=dev),
                  "v_norms": torch.empty(rows, device=dev),
                  "k_channels": torch.stack([chk[h][g] for h in range(Hh)]).to(torch.int32).contiguous(),
                  "v_channels": torch.stack([chv[h][g] for h in range(Hh)]).to(torch.int32).contiguous()}
            sk = torch.empty(max(tq.tq_workspace_bytes(pk[g], tq.TQ_OP_QUANTIZE, rows), 16), dtype=torch.uint8, device=dev)
            tq.tq_quantize_prod(pk[g], Xk, gd["k_idx"], gd["k_qjl"], gd["k_gamma"], gd["k_norms"], sk)
            tq.tq_quantize_mse(pv[g], Xv, gd["v_idx"], gd["v_norms"], sk)
            groups.append(gd)
        return groups

    def time_layers(groups, tokens, name):
        layer_bytes = sum(gd[key].numel() * gd[key].element_size() for gd in groups for key in code_keys)
        n_layers = max(4, min(64, int(math.ceil(0.9e9 / layer_bytes))))      # enough copies to exceed L2
        layers = [[{key: (val.clone() if key in code_keys else val) for key, val in gd.items()} for gd in groups]
                  for _ in range(n_layers)]
        ws_kv = torch.empty(tq.tq_attend_decode_workspace_bytes(2, Hh, tokens, grp), dtype=torch.uint8, device=dev)
        out_kv = torch.zeros((Hh * 4, hd), dtype=torch.float32, device=dev)

        def decode_all_layers():
            for lay in layers:
                tq.tq_attend_decode(lay, Hh, tokens, 4, Qc, 1.0 / math.sqrt(hd), out_kv, ws_kv)

        us_layer = time_call(decode_all_layers, name, min_ms=100.0, max_reps=20) * 1e3 / n_layers
        return {"tokens": tokens, "layers": n_layers, "us_per_layer": us_layer, "code_bytes_per_layer": layer_bytes,
                "codes_gbs": layer_bytes / (us_layer * 1e-6) / 1e9, "frac_hbm": layer_bytes / (us_layer * 1e-6) / 1e9 / peaks["hbm_gbs"]}

    base = time_layers(build_groups((3, 2), (3, 2), Tt), Tt, "c3:2.5bit")
    sweep = [time_layers(build_groups((3, 2), (3, 2), t), t, f"c3:len{t}") for t in (4096, 106496)]
    split35 = time_layers(build_groups((4, 3), (4, 3), Tt), Tt, "c3:3.5bit")
    return {"workload": f"c3: {Hh} KV heads x {Tt} tokens x {hd} channels (64 at 3 bits + 64 at 2 bits), K prod / V mse, 32 query heads",
            **base, "launches_per_layer": 3, "context_lengths": sweep,
            "split_3p5_bits": {"split": "64 channels at 4 bits + 64 at 3 bits", **split35}}


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_b200(a)
