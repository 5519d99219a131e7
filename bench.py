#!/usr/bin/env python
"""Benchmark of the fast-slow serving path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

A step is one pass of the whole cascade (features -> tree ensemble -> uncertainty
routing + compaction + wide-row gather -> slow model -> merge) over one batch of
seeded synthetic flows.  Rank 0 prints one JSON line.  The headline figures are those
of the configuration the metric is quoted on (config 2); on one GPU the same line
also carries, under "configs", the other four workloads (step time, per-kernel-class
times and rooflines, end-to-end figure from host memory, CPU-oracle baseline).  With
--impl reference the CPU oracle is timed instead (rank 0 only).  With N > 1 every
rank serves its own batch on its own GPU (flows are independent: no data-path
collective), and the only communication is the max of the elapsed times.
"""
import argparse
import dataclasses
import gc
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import flowgen  # noqa: E402

METRIC = "flows/s end-to-end on 1 B200; fast-path HBM GB/s and slow-path TC % of peak"
UNIT = "flows/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# the datasheet figures, for context beside every fraction of a measured peak
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
SM_COUNT, SM_MAX_MHZ = 148, 1965.0
# The tree walk is bound by the SM's load/store data pipe (one 128-byte wavefront per clock
# per SM), not by HBM.  Wavefronts a warp cannot do without IN THIS KERNEL'S NODE LAYOUT: per node
# visit one 64-bit node load (32 lanes x 8 B = 2 wavefronts) and one feature load (1); per tree the
# leaf payload (32 lanes x 4*C bytes, at 128 B per wavefront).  It is the floor of this layout, not
# of the method; node visits per second are printed beside it.
FOREST_WAVEFRONTS_PER_VISIT = 3
# DRAM bytes per launch measured with ncu for the dominant kernel class of a config, with the hash of the
# kernel's source at capture time: the figure turns null as soon as the kernel changes
# (profiles/gemm_traffic_config2_524288_flows.md).
TRAFFIC_BY_SOURCE = {("gemm", 2): {"src_hash": "159f94d817c7cda2", "bytes_per_row_per_launch": 1468544768 / 3 / 123679}}
PAPER_CONTEXT = ("paper: over 48.5k new flows/s on a 16-core CPU server; 76.3% of flows inferred in under 16 ms "
                 "(other hardware, real traffic; not comparable)")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def src_hash(name):
    p = os.path.join(ROOT, "paper_2402_03694_b200", "csrc", name)
    return hashlib.sha256(open(p, "rb").read()).hexdigest()[:16]


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                       "--format=csv,noheader,nounits", "-lms", "25"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.f.name)
        mhz, reasons, mx = [], set(), None
        for r in rows:
            r = [x.strip() for x in r]
            try:
                mhz.append(float(r[1]))
                mx = float(r[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if mhz:
            out.update(sm_mhz=float(np.median(mhz)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(mhz))
        return out


def device_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    return vis.split(",")[local] if vis else local


# ------------------------------------------------------------------------------------------------
def build_gpu_workload(cfg, n, rank, sf, hz, ctx, torch):
    """Inputs, models and threshold for one rank, using only the CUDA library for the
    method's arithmetic (feature sample for the split thresholds, validation scores
    for Algorithm 1)."""
    t0 = time.time()
    wide = flowgen.gen_packets(rank_data_seed(cfg, rank), n, cfg.P, cfg.H)
    fast = flowgen.fast_view(wide, cfg.N)
    t_gen = time.time() - t0
    fast_d = hz.upload_packets(fast, with_hdr=False)
    wide_d = hz.upload_packets(wide)
    m = min(n, 65536)
    feat = torch.empty((n, cfg.F), dtype=torch.float32, device="cuda")
    sf.sf_extract_features(ctx, fast_d["struct"], cfg.N, cfg.F, feat)
    feat_sample = feat[:m].cpu().numpy()
    forest_np = flowgen.gen_forest(cfg.seed_model, cfg.kind, cfg.T, cfg.depth, cfg.F, cfg.C, feat_sample, cfg.gbdt_sigma)
    forest = hz.make_forest(ctx, forest_np)
    if cfg.kind == "rf":
        nv = min(n, cfg.n_val)
        val = flowgen.gen_packets(cfg.seed_val, nv, cfg.N, 0)
        val_d = hz.upload_packets(val, with_hdr=False)
        fv = torch.empty((nv, cfg.F), dtype=torch.float32, device="cuda")
        pv = torch.empty((nv, cfg.C), dtype=torch.float32, device="cuda")
        sc = torch.empty(nv, dtype=torch.float32, device="cuda")
        ids = torch.empty(1, dtype=torch.uint32, device="cuda")
        ne = torch.empty(1, dtype=torch.uint32, device="cuda")
        sf.sf_extract_features(ctx, val_d["struct"], cfg.N, cfg.F, fv)
        sf.sf_fast_infer(ctx, forest, fv, nv, pv)
        never = hz.dev(np.full(cfg.C, 2.0, np.float32))
        sf.sf_route(ctx, sf.make_route_cfg(sf.SF_LC_GT, never, sf.SF_MLP16, sf.SF_BF16, cfg.P, 1), pv, nv, cfg.C,
                    None, ids, ne, None, None, None, sc)
        tau = np.full(cfg.C, sf.sf_universal_thresholds(sc.cpu().numpy(), [cfg.q_percent])[0], np.float32)
        sf.sf_ctx_poll(ctx, reset=True)
    else:
        tau = np.array([sf.SF_TAU_MARGIN_DEFAULT], np.float32)
    slow_np = flowgen.gen_mlp(cfg.seed_model, cfg.dims) if cfg.slow == "mlp" else flowgen.gen_cnn(cfg.seed_model, *cfg.cnn)
    slow = hz.make_slow(ctx, cfg, slow_np)
    del feat
    return {"wide": wide, "fast": fast, "wide_d": wide_d, "fast_d": fast_d, "forest": forest, "slow": slow,
            "tau": tau, "forest_np": forest_np, "slow_np": slow_np, "t_gen": t_gen}


def rank_data_seed(cfg, rank):
    """Every rank serves its own batch: flows are independent units, so ranks share nothing but the models."""
    return cfg.seed_data + 7919 * rank


def max_over_ranks(ms_local, dist, device):
    """The job's time is the slowest rank's (the only collective of the multi-GPU run)."""
    if dist is None:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_flows_per_s(world, flows_per_rank, steps, ms_total):
    return world * flows_per_rank * steps / (ms_total * 1e-3)


def hidden_flops_per_row(cfg):
    if cfg.slow == "mlp":
        return 2 * sum(cfg.dims[l] * cfg.dims[l + 1] for l in range(len(cfg.dims) - 2))
    L, Cin, C1, C2, k, _ = cfg.cnn
    return 2 * L * (k * Cin * C1 + k * C1 * C2)


def kernel_launches_per_step(cfg, capacity):
    """Kernels of this library that one sf_serve_batch call launches (the ncu launch lists under profiles/ agree)."""
    if cfg.slow == "mlp":
        slow = (len(cfg.dims) - 1) + (1 if cfg.slow_dtype == "f32" else 0)    # layers (+ argmax for fp32)
        nl = cfg.dims[-2]
        bn = 256 if nl % 256 == 0 else (128 if nl % 128 == 0 else 64)
        if cfg.slow_dtype == "bf16" and nl <= 1024 and nl // bn >= 2:
            slow -= 1                                                         # the head runs inside the last hidden layer's launch
    else:
        slow = 1                                                              # the fused CNN kernel
    return 1 + 1 + 3 + slow + 1          # extract, forest (takes the decisions itself), scan/scatter/gather, slow, merge


def tensor_peak_for(peaks, clocks):
    """The burst figure when the SM clock stayed at its maximum during the timed region (a short region), the
    sustained one when the clock had dropped under the power cap (a long one)."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if mhz and mx and mhz < 0.93 * mx:
        return peaks["bf16_tflops_sustained"], "sustained"
    return peaks["bf16_tflops"], "burst"


def rooflines_for(cfg, n, k_esc, avg, peaks, clocks):
    in_b = cfg.N * 6 + 4 * ((cfg.N + 31) // 32)
    per_esc_in = cfg.P * (6 + cfg.H) + 4 * ((cfg.P + 31) // 32) + 4
    esz = 2 if cfg.slow_dtype == "bf16" else 4
    Cf = cfg.C if cfg.kind == "rf" else 1
    tpeak, tkind = tensor_peak_for(peaks, clocks)
    work = {
        "extract": ("hbm", n * (in_b + 4 * cfg.F) / 1e9),
        "gather": ("hbm", k_esc * (per_esc_in + cfg.D * esz) / 1e9),
        # scan + scatter (the tree kernel's epilogue took the decisions): decision bytes in, ids out
        "score": ("hbm", (n + 4 * k_esc) / 1e9),
        # (binary boosted trees take the node of their two top levels from the constant bank: two 64-bit loads less per tree)
        "forest": ("alu", (n / 32.0) * cfg.T * (cfg.depth * FOREST_WAVEFRONTS_PER_VISIT - (4 if cfg.kind == "gbdt" and cfg.depth >= 2 and cfg.T <= 1024 else 0) +
                                               (4 * Cf * 32) / 128.0) / 1e9),
    }
    if cfg.slow_dtype == "bf16":
        work["gemm"] = ("tensor", k_esc * hidden_flops_per_row(cfg) / 1e12)
    else:
        work["gemm"] = ("fp32", k_esc * hidden_flops_per_row(cfg) / 1e12)
    if cfg.slow == "mlp" and cfg.slow_dtype == "bf16" and avg.get("head", 0.0) > 0:
        work["head"] = ("hbm", k_esc * (cfg.dims[-2] * esz + 4 * cfg.dims[-1]) / 1e9)       # reads the last hidden activations once
    out = {}
    for k, (bound, w) in work.items():
        ms = avg.get(k, 0.0)
        if ms <= 0:
            continue
        ach = w / (ms * 1e-3)
        if bound == "hbm":
            r = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                 "frac_of_nominal": ach / NOMINAL_PEAKS["hbm_gbs"]}
        elif bound == "tensor":
            r = {"bound": "tensor", "achieved": ach, "peak": tpeak, "unit": "TFLOP/s", "frac": ach / tpeak, "peak_kind": tkind,
                 "frac_of_burst": ach / peaks["bf16_tflops"], "frac_of_sustained": ach / peaks["bf16_tflops_sustained"],
                 "frac_of_nominal": ach / NOMINAL_PEAKS["bf16_tflops"]}
        elif bound == "fp32":
            pk = SM_COUNT * 128 * 2 * SM_MAX_MHZ * 1e6 / 1e12      # 128 FP32 lanes per SM, one FMA per lane and clock
            r = {"bound": "alu", "achieved": ach, "peak": pk, "unit": "TFLOP/s", "frac": ach / pk,
                 "peak_name": "fp32 FMA rate (148 SMs x 128 lanes x 2 flop x max SM clock)"}
        else:
            pk = SM_COUNT * SM_MAX_MHZ * 1e6 / 1e9
            r = {"bound": "alu", "achieved": ach, "peak": pk, "unit": "Gwavefront/s", "frac": ach / pk,
                 "peak_name": "this node layout's load/store wavefront floor (148 SMs x 1 wavefront/clk x max SM clock)",
                 "node_visits_per_s": n * cfg.T * cfg.depth / (ms * 1e-3)}
        r["ms"] = ms
        out[k] = r
    return out


# ---- the CPU oracle as a baseline ---------------------------------------------------------------
def oracle_stage_run(wl, threads):
    """The oracle's stages one after the other on the workload wl (tests/workload.make_workload), timed each."""
    import oracle
    cfg = wl["cfg"]
    t = [time.perf_counter()]
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=threads); t.append(time.perf_counter())
    fo = oracle.forest_infer(wl["forest"], feat, threads=threads); t.append(time.perf_counter())
    r = oracle.route_lc(fo, wl["tau"]) if cfg.kind == "rf" else oracle.route_absmargin(fo, float(np.asarray(wl["tau"]).ravel()[0]))
    t.append(time.perf_counter())
    bf16 = cfg.slow_dtype == "bf16"
    rows = oracle.wide_rows(0 if cfg.slow == "mlp" else 1, r["esc_ids"], wl["wide"], cfg.P, bf16, threads=threads)
    t.append(time.perf_counter())
    if cfg.slow == "mlp":
        _, ls = oracle.mlp(wl["slow"], rows, bf16, threads=threads)
    else:
        _, ls = oracle.cnn(wl["slow"], rows, bf16, threads=threads)
    t.append(time.perf_counter())
    oracle.merge(r["label"], r["esc_ids"], ls); t.append(time.perf_counter())
    names = ("extract", "forest", "route", "wide_rows", "slow", "merge")
    return {k: t[i + 1] - t[i] for i, k in enumerate(names)}, t[-1] - t[0], int(r["n_esc"])


def oracle_baseline(cfg, n, budget_s, threads):
    """Oracle (as it stands) on a bounded prefix of the workload: all host cores, then one core; per stage and in all.
    The sample sizes come from a small pilot run so that each leg takes about budget_s seconds."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from workload import make_workload

    def leg(th, pilot_n, budget):
        pn = min(n, pilot_n)
        wl = make_workload(dataclasses.replace(cfg, n=pn), n=pn, threads=threads)
        _, secs, _ = oracle_stage_run(wl, th)
        ns = int(min(n, max(pn, (budget / max(secs, 1e-6)) * pn)))
        ns = max(pn, (ns // 1024) * 1024) if ns >= 1024 else ns
        if ns > pn:
            wl = make_workload(dataclasses.replace(cfg, n=ns), n=ns, threads=threads)
        st, secs, esc = oracle_stage_run(wl, th)
        return ns, st, secs, esc

    ns, st, secs, esc = leg(threads, 4096, budget_s)
    n1, st1, secs1, esc1 = leg(1, 512, 0.6 * budget_s)
    return {"value": ns / secs, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "first %d flows of %s (%d assigned), all stages, %.1f s" % (ns, cfg.name, esc, secs),
            "per_stage_s": {k: round(v, 4) for k, v in st.items()},
            "one_core": {"value": n1 / secs1, "unit": UNIT, "cores": 1,
                         "sample": "first %d flows (%d assigned), %.1f s" % (n1, esc1, secs1),
                         "per_stage_s": {k: round(v, 4) for k, v in st1.items()}}}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from workload import make_workload
    threads = os.cpu_count() or 1
    n_sample = min(cfg.n, args.ref_flows)
    wl = make_workload(dataclasses.replace(cfg, n=n_sample), n=n_sample, threads=threads)
    times = []
    for i in range(args.warmup + args.steps + 1):                  # the first call is a warm-up too
        t0 = time.perf_counter()
        oracle.serve_batch(wl["cfg"], wl["fast"], wl["wide"], wl["forest"], wl["slow"], wl["tau"], threads=threads)
        dt = time.perf_counter() - t0
        if i > args.warmup:
            times.append(dt)
    total = sum(times)
    value = n_sample * len(times) / total
    sample = "first %d flows of config %d per step, all stages" % (n_sample, cfg.c)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "flows_per_step": n_sample, "note": "CPU oracle on a bounded sample"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- one batch configuration (1 to 4) -------------------------------------------------------------
def bench_batch(cfg, n, args, env, with_e2e, with_cpu, cpu_budget_s):
    """Times sf_serve_batch on config cfg; returns the figures of that config as a dict (rank 0), None on other ranks."""
    torch, sf, hz, ctx = env["torch"], env["sf"], env["hz"], env["ctx"]
    rank, world, local, dist = env["rank"], env["world"], env["local"], env["dist"]
    peaks = env["peaks"]
    wl = build_gpu_workload(cfg, n, rank, sf, hz, ctx, torch)
    cap = n
    rcfg = hz.route_cfg_for(cfg, hz.dev(wl["tau"], "cuda:%d" % local), cap)
    label = torch.zeros(n, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")

    def step():
        sf.sf_serve_batch(ctx, wl["forest"], wl["slow"], wl["fast_d"]["struct"], cfg.N, cfg.F, wl["wide_d"]["struct"],
                          rcfg, label, stage, n_esc)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    sf.sf_ctx_poll(ctx, reset=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index(local))
    sampler.start()
    time.sleep(0.3)
    # the timed region: K steps back to back, no per-kernel events (they cost time themselves)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), dist, torch.device("cuda", local))
    counters = sf.sf_ctx_poll(ctx, reset=True)
    k_esc = int(n_esc.cpu().numpy()[0])
    # where the time goes: a few more steps with the library's event ring on
    n_prof = max(3, min(args.steps, 8))
    sf.sf_ctx_set_timing(ctx, True)
    for _ in range(n_prof):
        step()
    torch.cuda.synchronize()
    recs = [sf.sf_ctx_get_timing(ctx, back) for back in range(n_prof)]
    sf.sf_ctx_set_timing(ctx, False)
    sf.sf_ctx_poll(ctx, reset=True)
    avg = {k: float(np.mean([r[k] for r in recs])) for k in recs[0]}
    ms_step = ms_total / args.steps
    value = whole_job_flows_per_s(world, n, args.steps, ms_total)
    if rank != 0:
        return None

    roof_all = rooflines_for(cfg, n, k_esc, avg, peaks, clocks)
    dom = max(roof_all, key=lambda k: roof_all[k]["ms"])
    src = {"gemm": "cnn.cu" if cfg.slow == "cnn" else "gemm_tc.cu", "forest": "forest.cu", "extract": "extract.cu",
           "gather": "route.cu", "score": "route.cu", "head": "gemm_tc.cu"}[dom]
    traffic = None
    tr = TRAFFIC_BY_SOURCE.get((dom, cfg.c))
    if tr is not None and tr["src_hash"] == src_hash(src):
        traffic = tr["bytes_per_row_per_launch"] * k_esc          # scaled by rows: traffic grows in proportion
    roofline = dict(roof_all[dom], kernel=dom, traffic=traffic, peak_source=env["peak_kind"],
                    launches_per_step=(len(cfg.dims) - 2) if dom == "gemm" and cfg.slow == "mlp" else 1)
    roofline.pop("ms")

    e2e = None
    if with_e2e:
        # end to end through the host-pointer entry point: pinned host planes, copies inside the timed region
        fast_h = hz.pinned_packets(wl["fast"], with_hdr=False)
        wide_h = hz.pinned_packets(wl["wide"])
        lab_h = torch.zeros(n, dtype=torch.uint8).pin_memory()
        st_h = torch.zeros(n, dtype=torch.uint8).pin_memory()
        ne_h = torch.zeros(1, dtype=torch.int32).pin_memory()
        rcfg_h = hz.route_cfg_for(cfg, np.ascontiguousarray(wl["tau"]), cap)

        def step_host():
            sf.sf_serve_batch_host(ctx, wl["forest"], wl["slow"], fast_h["struct"], cfg.N, cfg.F, wide_h["struct"],
                                   rcfg_h, lab_h, st_h, ne_h)
        for _ in range(2):
            step_host()
        n_calls = max(10, args.e2e_steps)
        t0 = time.perf_counter()
        for _ in range(n_calls):
            step_host()                                    # synchronous: returns when the labels are in host memory
        e2e_s = (time.perf_counter() - t0) / n_calls
        sf.sf_ctx_set_timing(ctx, True)                    # one more call, untimed, for where the time goes
        step_host()
        e2e_stages = {k: round(v, 4) for k, v in sf.sf_ctx_get_timing(ctx, 0).items() if v > 0}
        sf.sf_ctx_set_timing(ctx, False)
        # the library copies the fast planes of all flows, then only the assigned flows' wide rows
        h2d = sum(int(fast_h[k].numel() * fast_h[k].element_size()) for k in ("size", "iat_us", "dir_bits")) + \
            k_esc * (cfg.P * (6 + cfg.H) + 4 * ((cfg.P + 31) // 32)) + 4 * len(wl["tau"])
        e2e = {"value": world * n / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 2 * n + 4,
               "ms_per_step": e2e_s * 1e3, "calls": n_calls, "span_ms": e2e_stages,
               "note": "span_ms = first start to last end of each kernel class inside one call (classes overlap); "
                       "sf_serve_batch_host: pinned host planes in (fast planes copied up, the assigned flows' slow-context rows "
                       "read out of pinned memory by a kernel), labels out, synchronous; measured on rank 0"}
        assert np.array_equal(lab_h.numpy(), label.cpu().numpy())
        sf.sf_ctx_poll(ctx, reset=True)
        del fast_h, wide_h, lab_h, st_h

    out = {
        "ms_per_step": ms_step, "value": value, "unit": UNIT, "dtype": cfg.slow_dtype,
        "config": {"workload": cfg.name, "flows_per_gpu": n, "fast": "%s T=%d d=%d C=%d on %d pkts / %d feats" %
                   (cfg.kind, cfg.T, cfg.depth, cfg.C, cfg.N, cfg.F),
                   "slow": ("mlp " + "x".join(map(str, cfg.dims))) if cfg.slow == "mlp" else "cnn1d 128x8",
                   "assigned": k_esc, "assigned_frac": k_esc / n,
                   "l2": "inputs larger than L2 (%.2f GB of packet planes read per step)" %
                         (n * (cfg.P * (6 + cfg.H) + cfg.N * 6) / 1e9) if n * cfg.P * 19 > 2.0e8 else
                         "inputs smaller than L2 (%.1f MB): the step is launch-latency bound, nothing is flushed" %
                         (n * (cfg.P * (6 + cfg.H) + cfg.N * 6) / 1e6),
                   "parallelism": "replicas" if world > 1 else "single"},
        "per_stage_ms": avg,
        "per_stage_flows_per_s": {k: (n / (v * 1e-3) if v > 0 else None) for k, v in avg.items()},
        "per_stage_note": "per-kernel-class CUDA-event times from %d extra steps with the library's event ring on; "
                          "ms_per_step is from the timed region, ring off" % n_prof,
        "rooflines": roof_all, "roofline": roofline, "e2e": e2e,
        "gpu_launches": kernel_launches_per_step(cfg, cap) * args.steps, "clocks": clocks,
        "counters": {"n_flows": counters.n_flows, "n_escalated": counters.n_escalated,
                     "n_slow_done": counters.n_slow_done, "device_error": counters.device_error},
    }
    # release the device and pinned memory of this config before the CPU baseline and the next config
    sf.sf_slow_destroy(wl["slow"]); sf.sf_forest_destroy(wl["forest"])
    del wl, label, stage, n_esc, rcfg
    gc.collect()
    torch.cuda.empty_cache()
    out["cpu_baseline"] = oracle_baseline(cfg, n, cpu_budget_s, os.cpu_count() or 1) if with_cpu else None
    return out


# ---- the streaming configuration (5) --------------------------------------------------------------
def bench_stream(cfg, args, env, with_e2e, with_cpu, cpu_budget_s, steps):
    """Config 5: interleaved packets of many concurrent flows in 64K-packet batches through the
    device state table.  A step is `--batches-per-step` batches.  Reports first-seen flows/s,
    packets/s, answered flows/s and the share of answered flows that ended at the fast stage."""
    torch, sf, hz, ctx = env["torch"], env["sf"], env["hz"], env["ctx"]
    n_keys = args.flows or cfg.n
    m = 65536
    bps = args.batches_per_step
    prof_b = 8                                             # extra batches, run with the per-kernel timing ring on
    e2e_b = 32 if with_e2e else 0                          # extra batches, ingested from pinned host memory
    n_warm, n_meas = args.warmup * bps, steps * bps
    n_seq = n_meas                                         # the same number of batches once more, ingested without the pipelining
    n_batches = n_warm + n_meas + n_seq + prof_b + e2e_b
    log2_slots = max(10, int(np.ceil(np.log2(n_keys / 0.3))))
    src = flowgen.StreamSource(cfg.seed_data, n_keys, 1.1)
    # models of config 2 (forest on 8 packets with the 48-feature definition, 2048-wide MLP on 64 packets + zero padding)
    sample = flowgen.gen_packets(cfg.seed_data, 65536, cfg.N, 0)
    sd = hz.upload_packets(sample, with_hdr=False)
    feat = torch.empty((65536, cfg.F), dtype=torch.float32, device="cuda")
    sf.sf_extract_features(ctx, sd["struct"], cfg.N, cfg.F, feat)
    forest_np = flowgen.gen_forest(cfg.seed_model, "rf", cfg.T, cfg.depth, cfg.F, cfg.C, feat.cpu().numpy())
    forest = hz.make_forest(ctx, forest_np)
    pv = torch.empty((65536, cfg.C), dtype=torch.float32, device="cuda")
    sc = torch.empty(65536, dtype=torch.float32, device="cuda")
    ids = torch.empty(1, dtype=torch.uint32, device="cuda"); ne = torch.empty(1, dtype=torch.uint32, device="cuda")
    sf.sf_fast_infer(ctx, forest, feat, 65536, pv)
    never = hz.dev(np.full(cfg.C, 2.0, np.float32))
    sf.sf_route(ctx, sf.make_route_cfg(sf.SF_LC_GT, never, sf.SF_MLP16, sf.SF_BF16, 128, 1), pv, 65536, cfg.C, None, ids, ne,
                None, None, None, sc)
    tau = np.full(cfg.C, sf.sf_universal_thresholds(sc.cpu().numpy(), [cfg.q_percent])[0], np.float32)
    slow_np = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    slow = sf.sf_mlp_create(ctx, sf.SF_BF16, slow_np["dims"], slow_np["W"], slow_np["b"])
    sf.sf_ctx_poll(ctx, reset=True)
    slabs = min(n_keys, max(1 << 16, (n_batches * m) // 16))
    table = sf.sf_table_create(ctx, log2_slots, cfg.N, cfg.P, slabs)
    rcfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 128, 0, P_real=cfg.P)
    names = ("src", "dst", "sport", "dport", "proto", "dir", "size", "iat_us", "hdr")
    dev_batches, host_batches = [], []
    for b in range(n_batches):
        hb = src.batch(b, m)
        if b < n_batches - e2e_b:
            d = {k: hz.dev(hb[k]) for k in names}
            dev_batches.append(sf.make_pkt_batch(*[d[k] for k in names]))
        else:
            h = {k: torch.from_numpy(np.ascontiguousarray(hb[k])).pin_memory() for k in names}
            host_batches.append(sf.make_pkt_batch(*[h[k] for k in names]))
    res = torch.zeros((n_batches, 8), dtype=torch.int32, device="cuda")
    # the timed region: pipelined ingest (look-up + sort of batch b+1 under the model work of batch b), flushed before the
    # closing event so that every batch's work lies inside the region
    sf.sf_table_set_pipelined(ctx, table, True)
    for b in range(n_warm):
        sf.sf_table_ingest(ctx, table, dev_batches[b], forest, cfg.F, slow, rcfg, res[b])
    sf.sf_table_flush(ctx, table)
    torch.cuda.synchronize()
    b0 = n_warm
    sampler = ClockSampler(device_index(env["local"]))
    sampler.start(); time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for b in range(b0, b0 + n_meas):
        sf.sf_table_ingest(ctx, table, dev_batches[b], forest, cfg.F, slow, rcfg, res[b])
    sf.sf_table_flush(ctx, table)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    sf.sf_table_set_pipelined(ctx, table, False)
    c = sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    # for comparison, the following batches one after the other on one stream
    es0, es1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    es0.record()
    for b in range(b0 + n_meas, b0 + n_meas + n_seq):
        sf.sf_table_ingest(ctx, table, dev_batches[b], forest, cfg.F, slow, rcfg, res[b])
    es1.record()
    torch.cuda.synchronize()
    ms_seq = es0.elapsed_time(es1)
    sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    # per-kernel-class times from a few more batches with the event ring on (the events cost time themselves)
    sf.sf_ctx_set_timing(ctx, True)
    for b in range(b0 + n_meas + n_seq, b0 + n_meas + n_seq + prof_b):
        sf.sf_table_ingest(ctx, table, dev_batches[b], forest, cfg.F, slow, rcfg, res[b])
    torch.cuda.synchronize()
    recs = [sf.sf_ctx_get_timing(ctx, back) for back in range(prof_b)]
    sf.sf_ctx_set_timing(ctx, False)
    sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    stage_ms = {k: float(np.mean([x[k] for x in recs])) for k in recs[0]}
    r = res[b0:b0 + n_meas].cpu().numpy().astype(np.int64).sum(0)
    new_flows, fast_fired, fast_done, escalated, slow_fired, dropped, missed = [int(x) for x in r[:7]]
    secs = ms * 1e-3
    pk = n_meas * m
    answered = fast_done + slow_fired
    e2e = None
    if with_e2e:
        # the same stream continued from pinned host memory through the host-pointer call (copies up, counts back, synchronous)
        for hb in host_batches[:4]:
            sf.sf_table_ingest_host(ctx, table, hb, forest, cfg.F, slow, rcfg)
        t0 = time.perf_counter()
        nf = 0
        for hb in host_batches[4:]:
            nf += sf.sf_table_ingest_host(ctx, table, hb, forest, cfg.F, slow, rcfg).n_new_flows
        dt = time.perf_counter() - t0
        nb = len(host_batches) - 4
        e2e = {"value": nf / dt, "unit": "new flows/s", "packets_per_s": nb * m / dt, "us_per_batch": 1e6 * dt / nb,
               "h2d_bytes_per_step": bps * m * 33, "d2h_bytes_per_step": bps * 32, "calls": nb,
               "note": "sf_table_ingest_host per batch: nine pinned host planes copied up, counts back, synchronous"}
        sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    out = {"metric": "sustained new flows/s through the device state table (config 5)", "value": new_flows / secs,
           "unit": "new flows/s", "ms_per_step": ms / steps, "dtype": "bf16",
           "config": {"workload": cfg.name, "keys": n_keys, "log2_slots": log2_slots, "batch_packets": m,
                      "batches_per_step": bps, "steps": steps, "zipf": 1.1, "l2": "state table larger than L2 (%.1f GB)" %
                      ((1 << log2_slots) * (31 + cfg.N * 19 + 4) / 1e9)},
           "packets_per_s": pk / secs, "answered_flows_per_s": answered / secs,
           "fraction_answered_at_fast_stage": (fast_done / answered) if answered else None,
           "counts": {"new_flows": new_flows, "fast_fired": fast_fired, "fast_done": fast_done, "escalated": escalated,
                      "slow_fired": slow_fired, "dropped_after_decision": dropped, "missed": missed},
           "per_batch_stage_ms": stage_ms, "us_per_batch": 1e3 * ms / n_meas, "us_per_batch_unpipelined": 1e3 * ms_seq / n_seq,
           "pipelined": "sf_table_set_pipelined: look-up and sort of batch b+1 on the caller's stream under the model work of batch b on "
                        "the table's stream; flushed inside the timed region",
           "launches_per_batch": STREAM_LAUNCHES_PER_BATCH, "gpu_launches": STREAM_LAUNCHES_PER_BATCH * n_meas,
           "sector_traffic_gbs": pk * 200 / secs / 1e9,
           "e2e": e2e, "clocks": clocks, "device_error": c.device_error}
    sf.sf_table_destroy(table); sf.sf_slow_destroy(slow); sf.sf_forest_destroy(forest)
    del dev_batches, host_batches, res
    gc.collect()
    torch.cuda.empty_cache()
    if with_cpu:
        out["cpu_baseline"] = oracle_stream_baseline(cfg, n_keys, m, cpu_budget_s)
    return out


STREAM_LAUNCHES_PER_BATCH = 13


def oracle_stream_baseline(cfg, n_keys, m, budget_s):
    """The packet-by-packet reference (oracle/stream.py, pure Python) on the first batches of the same stream."""
    import oracle
    from oracle.stream import simulate_stream
    threads = os.cpu_count() or 1
    sample = flowgen.gen_packets(cfg.seed_data, 65536, cfg.N, 0)
    feat = oracle.extract_features(sample, cfg.N, cfg.F, threads=threads)
    forest = flowgen.gen_forest(cfg.seed_model, "rf", cfg.T, cfg.depth, cfg.F, cfg.C, feat)
    u = oracle.route_lc(oracle.forest_infer(forest, feat, threads=threads), 2.0)["score"]
    tau = np.full(cfg.C, oracle.universal_thresholds(u, [cfg.q_percent])[0], np.float32)
    slow = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    src = flowgen.StreamSource(cfg.seed_data, n_keys, 1.1)
    b0 = src.batch(0, 8192)
    t0 = time.perf_counter()
    simulate_stream([b0], cfg.N, cfg.P, cfg.F, forest, tau, slow, 128, True, threads=threads)
    pilot = time.perf_counter() - t0
    nb = int(max(1, min(8, budget_s / max(pilot * 8, 1e-6))))
    batches = [src.batch(b, m) for b in range(nb)]
    t0 = time.perf_counter()
    _, cnt = simulate_stream(batches, cfg.N, cfg.P, cfg.F, forest, tau, slow, 128, True, threads=threads)
    dt = time.perf_counter() - t0
    return {"value": cnt["new_flows"] / dt, "unit": "new flows/s", "packets_per_s": nb * m / dt, "cores": 1, "kind": "oracle",
            "sample": "first %d batches of %d packets of the same stream, sequential dictionary pass in Python "
                      "(model stages on %d threads), %.1f s" % (nb, m, threads, dt)}


def slow_model_sustained(cfg, seconds, env):
    """Diagnostic, not a bench line: the slow model alone, back to back for `seconds`, with the SM clock and the board power
    sampled every 25 ms - shows what the tensor pipe sustains under the power limit next to a short burst."""
    torch, sf, hz, ctx = env["torch"], env["sf"], env["hz"], env["ctx"]
    if cfg.slow != "mlp" or cfg.slow_dtype != "bf16":
        raise SystemExit("--slow-sustained: a bf16 MLP config (2, 3 or 5)")
    rows_n = int(min(cfg.n, 4_000_000) * ((100 - cfg.q_percent) / 100.0 if cfg.q_percent else 0.3))   # about the assigned share
    model = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    h = sf.sf_mlp_create(ctx, sf.SF_BF16, model["dims"], model["W"], model["b"])
    g = torch.Generator(device="cuda").manual_seed(cfg.seed_data)
    x = (torch.randn(rows_n, cfg.dims[0], device="cuda", generator=g) * 0.5).to(torch.bfloat16)
    nd = torch.tensor([rows_n], dtype=torch.int32, device="cuda")
    logits = torch.zeros(rows_n, cfg.dims[-1], device="cuda")
    lab = torch.zeros(rows_n, dtype=torch.uint8, device="cuda")
    flops = rows_n * hidden_flops_per_row(cfg)
    for _ in range(3):
        sf.sf_slow_infer(ctx, h, x, nd, rows_n, logits, lab)
    torch.cuda.synchronize()
    time.sleep(1.0)
    f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
    p = subprocess.Popen(["nvidia-smi", "-i", str(env["local"]), "--query-gpu=clocks.sm,power.draw,clocks_event_reasons.sw_power_cap",
                          "--format=csv,noheader,nounits", "-lms", "25"], stdout=f, stderr=subprocess.DEVNULL)
    ev = [torch.cuda.Event(enable_timing=True)]
    ev[0].record()
    t0 = time.perf_counter()
    while time.perf_counter() - t0 < seconds and len(ev) < 20000:
        for _ in range(10):
            sf.sf_slow_infer(ctx, h, x, nd, rows_n, logits, lab)
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        ev.append(e)
        if len(ev) % 8 == 0:
            ev[-1].synchronize()                            # keep the launch queue short so that the wall clock bounds the loop
    torch.cuda.synchronize()
    p.terminate()
    p.wait()
    ms = np.array([ev[i].elapsed_time(ev[i + 1]) / 10 for i in range(len(ev) - 1)])
    rows = [r.split(",") for r in open(f.name).read().strip().splitlines() if r.count(",") >= 2]
    os.unlink(f.name)
    half = rows[len(rows) // 2:]
    out = {"diagnostic": "slow model alone, back to back", "workload": cfg.name, "rows": rows_n, "seconds": seconds,
           "forwards": 10 * (len(ev) - 1), "first_10_forwards_tflops": flops / ms[0] / 1e9,
           "second_half_tflops": flops / float(np.mean(ms[len(ms) // 2:])) / 1e9,
           "second_half_sm_mhz_median": float(np.median([float(r[0]) for r in half])) if half else None,
           "second_half_power_w_median": float(np.median([float(r[1]) for r in half])) if half else None,
           "sw_power_cap_active_share": float(np.mean([r[2].strip().lower().startswith("active") for r in rows])) if rows else None}
    sf.sf_slow_destroy(h)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="the headline workload (default: the one the metric is quoted on)")
    ap.add_argument("--flows", type=int, default=0, help="override flows per batch (0 = the config's)")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--ref-flows", type=int, default=4096)
    ap.add_argument("--cpu-budget", type=float, default=8.0, help="seconds of oracle time for the headline config's all-core leg")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="only the headline config (no `configs` object)")
    ap.add_argument("--batches-per-step", type=int, default=16)
    ap.add_argument("--slow-sustained", type=float, default=0.0,
                    help="diagnostic: loop the config's bf16 MLP alone for this many seconds and print clocks, power and TFLOP/s")
    args = ap.parse_args()
    cfg = flowgen.get_config(args.config)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2402_03694_b200 import build as sfbuild
    if rank == 0:
        sfbuild.build()
    if dist is not None:
        dist.barrier()
    from paper_2402_03694_b200 import binding as sf, harness as hz
    ctx = sf.sf_ctx_create(local, 0)
    peaks, peak_kind = load_peaks()
    env = {"torch": torch, "sf": sf, "hz": hz, "ctx": ctx, "rank": rank, "world": world, "local": local, "dist": dist,
           "peaks": peaks, "peak_kind": peak_kind}
    if args.slow_sustained > 0:
        if rank == 0:
            print(json.dumps(slow_model_sustained(cfg, args.slow_sustained, env)))
        return
    t_start = time.time()
    with_e2e, with_cpu = not args.no_e2e, not args.no_cpu_baseline
    if cfg.c == 5:
        head = bench_stream(cfg, args, env, with_e2e, with_cpu, args.cpu_budget, args.steps)
    else:
        head = bench_batch(cfg, args.flows or cfg.n, args, env, with_e2e, with_cpu, args.cpu_budget)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {"metric": head.pop("metric", METRIC), "value": head.pop("value"), "unit": head.pop("unit"), "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": head.pop("ms_per_step"), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": head.pop("dtype"), "data": "synthetic"}
    line.update(head)
    # the other four workloads, one GPU only (under torchrun the GPUs are held for the headline alone)
    if world == 1 and not args.no_others and not args.flows and cfg.c == 2:
        others = {}
        for c in (1, 3, 4, 5):
            oc = flowgen.get_config(c)
            try:
                if c == 5:
                    o = bench_stream(oc, args, env, with_e2e, with_cpu, 0.4 * args.cpu_budget, min(args.steps, 10))
                else:
                    o = bench_batch(oc, oc.n, args, env, with_e2e, with_cpu, 0.4 * args.cpu_budget)
            except Exception as e:                                  # one failing workload must not hide the others
                o = {"error": "%s: %s" % (type(e).__name__, e)}
            others[oc.name] = o
        line["configs"] = others
    line["bench_wall_s"] = round(time.time() - t_start, 1)
    line["context"] = PAPER_CONTEXT
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
