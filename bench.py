#!/usr/bin/env python
"""Benchmark of the gf.apply hot path on B200: interactions/s and roofline fractions.

One *step* is one pass of the whole hot path over one batch of seeded synthetic input:
  CSR relation   (R-MAT scale 20, 16.8M directed edges, F=64 fp32): sum forward, sum backward
                 (grad x, grad w), max forward, max backward, degree histogram;
  radius relation (1M uniform points, periodic unit cube, 32 expected neighbours, F=32):
                 cell binning + fused Gaussian forward, backward (grad x, grad positions);
  Lennard-Jones   (160^3 jittered lattice, cutoff 2.5): cell binning + fused force/energy.
One interaction = one directed edge / one ordered accepted pair visited by one traversal.

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line (rank 0).  Under
torchrun every rank runs an independent replica of the step on its own GPU (the path has no
exchange step); the time is the max over ranks and `value` the sum of all ranks' work.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workloads.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "interactions/sec fwd and fwd+bwd for gf.apply"
UNIT = "interactions/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self.stop_flag.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.02)

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------ workloads
def make_workloads(seed):
    t0 = time.time()
    w = {"csr": gen.config("cfg1", seed), "rad": gen.config("cfg2", seed), "lj": gen.config("cfg3", seed)}
    w["gen_seconds"] = time.time() - t0
    return w


def roofline_models(w, counts, hbm_gbs, clock_mhz):
    """Algorithmic work per launch of every row of the hot path.

    CSR: cache-oblivious gather model, bytes = E (col + w + one source row) + N (rowptr + one
    output row); backward adds the cotangent row, the atomic read-modify-write of the
    source-gradient row and the edge gradient.  Radius: fp32 lane operations (FMA = 1),
    7 per candidate pair (27-cell stencil) plus F+3 (Gaussian forward), 3F+12 (Gaussian
    backward) or 14 (Lennard-Jones) per accepted pair.
    """
    c = w["csr"]
    E, N, F = c["E"], c["n"], c["F"]
    fb = 4 * F
    m = {}
    m["csr_sum_fwd"] = dict(bound="hbm", work=E * (8 + fb) + N * (4 + fb), inter=E)
    m["csr_max_fwd"] = dict(bound="hbm", work=E * (8 + fb) + N * (4 + 2 * fb), inter=E)
    m["csr_sum_bwd"] = dict(bound="hbm", work=E * (8 + fb + 4 + 2 * fb) + N * (4 + fb) + N * fb, inter=E)
    m["csr_max_bwd"] = dict(bound="hbm", work=N * F * (4 + 4 + 4 + 4 + 4 + 8 + 8), inter=E)
    m["csr_hist"] = dict(bound="hbm", work=4 * (N + 1), inter=0)
    alu_peak = 148 * 128 * clock_mhz * 1e6      # fp32 lane operations per second
    for key, cfg, acc in (("rad", w["rad"], counts["rad_pairs"]), ("lj", w["lj"], counts["lj_pairs"])):
        n = cfg["n"]
        ncell = counts[key + "_ncell"]
        cand = 27.0 * n * n / ncell             # candidate pairs tested by a 27-cell stencil
        if key == "rad":
            Fr = cfg["F"]
            m["radius_gauss_fwd"] = dict(bound="alu", work=7 * cand + (Fr + 3) * acc, inter=acc)
            m["radius_gauss_bwd"] = dict(bound="alu", work=7 * cand + (3 * Fr + 12) * acc, inter=acc)
        else:
            m["radius_lj_fwd"] = dict(bound="alu", work=7 * cand + 14 * acc, inter=acc)
    for k, v in m.items():
        v["peak"] = hbm_gbs * 1e9 if v["bound"] == "hbm" else alu_peak
    return m


def combine_ranks(dist, device, total_ms, e2e_ms, interactions):
    """Replicas only: the step time of the job is the slowest rank's, the work is the sum."""
    import torch
    if dist is None:
        return total_ms, e2e_ms, float(interactions)
    t = torch.tensor([total_ms, e2e_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tot = torch.tensor([float(interactions)], device=device, dtype=torch.float64)
    dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    return t[0].item(), t[1].item(), tot.item()


# DRAM traffic per unit measured with ncu on reduced replicas (profiles/*.md), used to scale
# `roofline.traffic` to a full launch: bytes per particle / point / edge of one launch.
TRAFFIC_PER_UNIT = {
    "radius_lj_fwd": ("particle", 48.4),          # profiles/radius_lj_pairs_1M.md: 32.4 B measured + the 16-byte row that leaves L2 at full size
    "radius_gauss_fwd": ("point", 186.7),         # profiles/radius_traverse_gaussian_300k.md
    "radius_gauss_bwd": ("point", 364.6),
    "csr_sum_fwd": ("edge", 21.1),                # profiles/csr_kernels_rmat_scale18.md
    "csr_sum_bwd": ("edge", 45.3),
    "csr_max_bwd": ("edge", 52.1),
}


# ------------------------------------------------------------------------------ our arm
def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2609_24802_b200 import api as T

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    hbm_gbs, sm_max, peak_kind = measured_peaks()
    w = make_workloads(args.seed + rank)
    c, r, lj = w["csr"], w["rad"], w["lj"]

    def pin(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

    # pinned host copies (for the end-to-end leg) and device-resident inputs
    h = {"rowptr": pin(c["rowptr"]), "col": pin(c["col"]), "w": pin(c["w"]), "x": pin(c["x"]), "gy": pin(c["gy"]),
         "rpos": pin(r["pos"]), "rx": pin(r["x"]), "rgy": pin(r["gy"]), "ljpos": pin(lj["pos"])}
    d = {k: v.to(dev) for k, v in h.items()}
    g = T.CsrRelation(d["rowptr"], d["col"], c["n"])
    N, E, F = c["n"], c["E"], c["F"]
    n2, F2 = r["n"], r["F"]
    n3 = lj["n"]

    out_sum = torch.empty((N, F), device=dev); out_max = torch.empty((N, F), device=dev)
    arg = torch.empty((N, F), dtype=torch.int32, device=dev)
    gx = torch.empty((N, F), device=dev); gw = torch.empty(E, device=dev)
    gxm = torch.empty((N, F), device=dev); gwm = torch.empty(E, device=dev)
    ws_csr = torch.empty(T.tiga_csr_workspace_bytes(g, F, T.F32, T.MAX), dtype=torch.uint8, device=dev)
    rout = torch.empty((n2, F2), device=dev); rcount = torch.empty(n2, dtype=torch.int32, device=dev)
    rgx = torch.empty((n2, F2), device=dev); rgp = torch.empty((n2, 3), device=dev)
    ws_rad = torch.empty(T.tiga_radius_workspace_bytes(n2, F2, r["r"], r["box"], r["periodic"]), dtype=torch.uint8, device=dev)
    ljout = torch.empty((n3, 4), device=dev); ljcount = torch.empty(n3, dtype=torch.int32, device=dev)
    ws_lj = torch.empty(T.tiga_radius_workspace_bytes(n3, 4, lj["r"], lj["box"], lj["periodic"]), dtype=torch.uint8, device=dev)

    rows = ["csr_sum_fwd", "csr_sum_bwd", "csr_max_fwd", "csr_max_bwd", "csr_hist",
            "radius_gauss_fwd", "radius_gauss_bwd", "radius_lj_fwd"]
    stream = torch.cuda.current_stream()

    # the step in its three independent parts (cfg1 CSR, cfg2 radius, cfg3 Lennard-Jones)
    def part_csr(mark):
        T.tiga_apply_csr(g, d["x"], d["w"], T.SUM, out=out_sum, ws=ws_csr); mark(1)
        T.tiga_apply_csr_backward(g, d["x"], d["w"], d["gy"], T.SUM, grad_x=gx, grad_w=gw); mark(2)
        T.tiga_apply_csr(g, d["x"], d["w"], T.MAX, out=out_max, argmax=arg, ws=ws_csr); mark(3)
        T.tiga_apply_csr_backward(g, d["x"], d["w"], d["gy"], T.MAX, argmax=arg, grad_x=gxm, grad_w=gwm); mark(4)
        hist, mx = T.tiga_csr_degree_histogram(g, 4096); mark(5)
        return hist, mx

    def part_radius(mark):
        T.tiga_apply_radius(d["rpos"], d["rx"], r["r"], r["box"], r["periodic"], T.MSG_GAUSS, p0=r["sigma"],
                            out=rout, count=rcount, ws=ws_rad); mark(6)
        T.tiga_apply_radius_backward(d["rpos"], d["rx"], d["rgy"], r["r"], r["box"], r["periodic"], r["sigma"],
                                     ws=ws_rad, reuse_plan=True, grad_feat=rgx, grad_pos=rgp); mark(7)

    def part_lj(mark):
        # forces and energies only, as the row is defined; the pair count of the metric comes from one
        # counting call before the timed region
        T.tiga_apply_radius(d["ljpos"], None, lj["r"], lj["box"], lj["periodic"], T.MSG_LJ, p0=lj["eps"], p1=lj["s"],
                            out=ljout, ws=ws_lj); mark(8)

    def step(ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record(stream)
        mark(0)
        hist, mx = part_csr(mark)
        part_radius(mark)
        part_lj(mark)
        return hist, mx

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    T.tiga_apply_radius(d["ljpos"], None, lj["r"], lj["box"], lj["periodic"], T.MSG_LJ, p0=lj["eps"], p1=lj["s"],
                        out=ljout, count=ljcount, ws=ws_lj)
    for _ in range(max(args.warmup, 3)):
        step()
    sync_all()
    counts = {"rad_pairs": int(rcount.sum().item()), "lj_pairs": int(ljcount.sum().item()),
              "rad_ncell": int(np.prod(T.tiga_radius_grid(n2, r["r"], r["box"], r["periodic"])[0])),
              "lj_ncell": int(np.prod(T.tiga_radius_grid(n3, lj["r"], lj["box"], lj["periodic"])[0]))}
    inter_step = 4 * E + 2 * counts["rad_pairs"] + counts["lj_pairs"]

    # ---- timed region: device-resident inputs
    sampler = ClockSampler(physical_gpu_index(local_rank))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(9)] for _ in range(args.steps)]
    l0 = T.launch_count()
    sync_all()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(args.steps):
        step(evs[k])
    t_end.record(stream)
    sync_all()
    sampler.stop_flag.set()
    launches = T.launch_count() - l0
    total_ms = t_start.elapsed_time(t_end)
    per_row_ms = [statistics.mean(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(8)]
    clocks = sampler.summary()

    # ---- end-to-end leg: inputs start in pinned host memory, results end in pinned host memory
    res_h = {"out_sum": torch.empty((N, F)).pin_memory(), "gx": torch.empty((N, F)).pin_memory(),
             "gw": torch.empty(E).pin_memory(), "out_max": torch.empty((N, F)).pin_memory(),
             "gxm": torch.empty((N, F)).pin_memory(), "gwm": torch.empty(E).pin_memory(),
             "hist": torch.empty(4096, dtype=torch.int64).pin_memory(),
             "rout": torch.empty((n2, F2)).pin_memory(), "rgx": torch.empty((n2, F2)).pin_memory(),
             "rgp": torch.empty((n2, 3)).pin_memory(), "ljout": torch.empty((n3, 4)).pin_memory()}
    h2d = sum(v.numel() * v.element_size() for v in h.values())
    d2h = sum(v.numel() * v.element_size() for v in res_h.values())

    # Three streams: inputs go up on one, kernels run on the bench stream, results come down on a third,
    # so that the copies of one part overlap the kernels and the copies of the others (PCIe is full
    # duplex).  Events order every buffer: inputs are overwritten only after the kernels that read
    # them, outputs only after their copy to the host.  All of it lies inside the timed region.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    parts = {
        "csr": (["rowptr", "col", "w", "x", "gy"], part_csr,
                lambda hist: [("out_sum", out_sum), ("gx", gx), ("gw", gw), ("out_max", out_max), ("gxm", gxm), ("gwm", gwm), ("hist", hist)]),
        "radius": (["rpos", "rx", "rgy"], lambda mark: part_radius(mark), lambda _: [("rout", rout), ("rgx", rgx), ("rgp", rgp)]),
        "lj": (["ljpos"], lambda mark: part_lj(mark), lambda _: [("ljout", ljout)]),
    }
    computed = {k: None for k in parts}      # events of the previous step
    drained = {k: None for k in parts}

    def e2e_step():
        for name, (inputs, compute, outputs) in parts.items():
            if computed[name] is not None:
                s_in.wait_event(computed[name])
            with torch.cuda.stream(s_in):
                for k in inputs:
                    d[k].copy_(h[k], non_blocking=True)
                up = torch.cuda.Event(); up.record(s_in)
            stream.wait_event(up)
            if drained[name] is not None:
                stream.wait_event(drained[name])
            res = compute(lambda i: None)
            hist = res[0] if isinstance(res, tuple) else None
            done = torch.cuda.Event(); done.record(stream)
            computed[name] = done
            s_out.wait_event(done)
            with torch.cuda.stream(s_out):
                for k, src in outputs(hist):
                    res_h[k].copy_(src, non_blocking=True)
                    src.record_stream(s_out)
                dn = torch.cuda.Event(); dn.record(s_out)
            drained[name] = dn

    def e2e_join():
        for ev in drained.values():
            if ev is not None:
                stream.wait_event(ev)

    e2e_step()
    e2e_join()
    sync_all()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e2e_join()
    e1.record(stream)
    sync_all()
    e2e_ms = e0.elapsed_time(e1)

    total_ms, e2e_ms, inter_all = combine_ranks(dist, dev, total_ms, e2e_ms, inter_step)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = inter_all / (ms_per_step * 1e-3)
    clock_for_alu = clocks["sm_mhz"] or sm_max
    models = roofline_models(w, counts, hbm_gbs, clock_for_alu)
    row_report = {}
    for name, ms in zip(rows, per_row_ms):
        mdl = models[name]
        ach = mdl["work"] / (ms * 1e-3)
        row_report[name] = {"ms": round(ms, 4), "interactions_per_s": (mdl["inter"] / (ms * 1e-3)) if mdl["inter"] else None,
                            "bound": mdl["bound"],
                            "achieved": ach / (1e9 if mdl["bound"] == "hbm" else 1e12),
                            "peak": mdl["peak"] / (1e9 if mdl["bound"] == "hbm" else 1e12),
                            "unit": "GB/s" if mdl["bound"] == "hbm" else "Tlaneop/s", "frac": ach / mdl["peak"]}
    dom = max(rows, key=lambda k: row_report[k]["ms"])
    dr = row_report[dom]
    units = {"particle": n3, "point": n2, "edge": E}
    traffic = None
    if dom in TRAFFIC_PER_UNIT:
        kind, per = TRAFFIC_PER_UNIT[dom]
        traffic = per * units[kind]
    fwd = {"csr_sum": E / (per_row_ms[0] * 1e-3), "csr_max": E / (per_row_ms[2] * 1e-3),
           "radius_gauss": counts["rad_pairs"] / (per_row_ms[5] * 1e-3), "radius_lj": counts["lj_pairs"] / (per_row_ms[7] * 1e-3)}
    fwd_bwd = {"csr_sum": E / ((per_row_ms[0] + per_row_ms[1]) * 1e-3), "csr_max": E / ((per_row_ms[2] + per_row_ms[3]) * 1e-3),
               "radius_gauss": counts["rad_pairs"] / ((per_row_ms[5] + per_row_ms[6]) * 1e-3)}

    # ---- the stored-relation forward in detail: three bandwidth fractions, the L2 gather ceiling,
    #      warm and flushed L2 (outside the timed step; rank 0 only)
    def timed(fn, reps=10, before=None):
        ts = []
        for _ in range(reps):
            if before is not None:
                before()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    gen_t = torch.Generator(device=dev); gen_t.manual_seed(args.seed)
    table = torch.randn((60 * 2**20 // (4 * F), F), device=dev, generator=gen_t)              # 60 MiB of 256-byte rows: fits L2
    ridx = torch.randint(0, table.shape[0], (E,), device=dev, generator=gen_t, dtype=torch.int32)
    sink = torch.zeros(1, device=dev)
    for _ in range(3):
        T.tiga_probe_row_gather(table, ridx, sink)
    t_l2 = timed(lambda: T.tiga_probe_row_gather(table, ridx, sink))
    t_col = timed(lambda: T.tiga_probe_row_gather(d["x"], d["col"], sink))                 # the workload's own index stream and table
    l2_peak = E * 4.0 * F / (t_l2 * 1e-3)
    flush_buf = torch.empty(512 * 2**20, dtype=torch.uint8, device=dev)
    fwd_call = lambda: T.tiga_apply_csr(g, d["x"], d["w"], T.SUM, out=out_sum, ws=ws_csr)
    t_warm = timed(fwd_call)
    t_cold = timed(fwd_call, before=lambda: flush_buf.zero_())
    touched = int(torch.unique(d["col"]).numel())
    t_fwd = per_row_ms[0]
    b_min = 4.0 * (N + 1) + 8.0 * E + 4.0 * F * touched + 4.0 * F * N
    b_dram = TRAFFIC_PER_UNIT["csr_sum_fwd"][1] * E
    csr_detail = {
        "row": "csr_sum_fwd", "ms_in_step": round(t_fwd, 4), "ms_back_to_back_warm_l2": round(t_warm, 4),
        "ms_l2_flushed_512MiB_write_between_calls": round(t_cold, 4),
        "f_alg": row_report["csr_sum_fwd"]["frac"], "f_dram": b_dram / (t_fwd * 1e-3) / (hbm_gbs * 1e9),
        "f_min": b_min / (t_fwd * 1e-3) / (hbm_gbs * 1e9),
        "bytes_alg": models["csr_sum_fwd"]["work"], "bytes_dram_ncu_scaled": b_dram, "bytes_min": b_min, "touched_source_rows": touched,
        "l2_gather_peak_GBps": l2_peak / 1e9,
        "l2_gather_peak_note": "tiga_probe_row_gather: 16.8M uniform random 256-byte row gathers from a 60 MiB table",
        "gather_of_own_index_stream_ms": round(t_col, 4),
        "T_l2roof_over_T": (E * 4.0 * F / l2_peak) / (t_fwd * 1e-3),
        "T_own_gather_over_T": t_col / t_fwd,
    }
    del table, ridx, flush_buf

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "cfg1 CSR R-MAT scale 20 E=16,777,216 F=64 fp32 (sum fwd+bwd, max fwd+bwd, degree histogram) "
                               "+ cfg2 radius N=1,000,000 periodic F=32 Gaussian (bin+fwd, bwd) "
                               "+ cfg3 Lennard-Jones N=4,096,000 (bin+fwd)",
                   "seed": args.seed, "l2": "inputs larger than L2 (644 MB CSR inputs; each kernel streams >126 MB between repeats)",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "interactions_per_step": inter_step, "radius_pairs": counts["rad_pairs"], "lj_pairs": counts["lj_pairs"],
                   "lj_pairs_note": "counted by one call with neighbour counts before the timed region; the timed Lennard-Jones call returns forces and energies only"},
        "fwd_interactions_per_s": fwd, "fwd_bwd_interactions_per_s": fwd_bwd, "rows": row_report,
        "roofline": {"kernel": dom, "bound": dr["bound"], "achieved": dr["achieved"], "peak": dr["peak"], "unit": dr["unit"],
                     "frac": dr["frac"], "traffic": traffic,
                     "traffic_note": "ncu dram bytes of this kernel on a reduced replica, scaled by units processed (profiles/)",
                     "peak_source": peak_kind + (" hbm copy" if dr["bound"] == "hbm" else
                                                                                     " 148 SM x 128 lanes x sampled SM clock")},
        "e2e": {"value": inter_all / (e2e_ms / args.steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches, "clocks": clocks, "csr_detail": csr_detail,
    }
    if not args.no_cpu_baseline and world >= 1:
        line["cpu_baseline"] = cpu_baseline(w, seconds_hint=20)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ CPU oracle arms
def cpu_baseline(w, seconds_hint=20):
    """The fp64 oracle, as it stands, on a bounded sample of the step's workloads."""
    import oracle
    c = w["csr"]
    t0 = time.time()
    _, _, arg = oracle.csr_forward(c["rowptr"], c["col"], c["x"], c["w"], oracle.MAX)
    oracle.csr_forward(c["rowptr"], c["col"], c["x"], c["w"], oracle.SUM)
    oracle.csr_backward_sum(c["rowptr"], c["col"], c["x"], c["w"], c["gy"])
    oracle.csr_backward_max(c["rowptr"], c["col"], c["x"], c["w"], c["gy"], arg)
    oracle.degree_histogram(c["rowptr"], 4096)
    t_csr = time.time() - t0
    rr = w["rad"]
    t0 = time.time()
    _, _, cnt = oracle.radius_forward(rr["pos"], rr["x"], rr["r"], rr["box"], rr["periodic"], oracle.MSG_GAUSS,
                                      p0=rr["sigma"], use_cells=True)
    oracle.radius_backward_gauss(rr["pos"], rr["x"], rr["gy"], rr["r"], rr["box"], rr["periodic"], rr["sigma"], use_cells=True)
    t_rad = time.time() - t0
    lj = w["lj"]
    t0 = time.time()
    _, _, cnt3 = oracle.radius_forward(lj["pos"], None, lj["r"], lj["box"], lj["periodic"], oracle.MSG_LJ, 1.0, 1.0, use_cells=True)
    t_lj = time.time() - t0
    inter = 4 * c["E"] + 2 * int(cnt.sum()) + int(cnt3.sum())
    return {"value": inter / (t_csr + t_rad + t_lj), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"the whole step once: cfg1 CSR sum and max fwd + bwd and the histogram (4 x {c['E']} edges, {t_csr:.1f} s) + cfg2 radius Gaussian "
                      f"fwd+bwd with the oracle's cell directory (2 x {int(cnt.sum())} pairs, {t_rad:.1f} s) + cfg3 "
                      f"Lennard-Jones with the cell directory ({int(cnt3.sum())} pairs, {t_lj:.1f} s)"}


def run_reference(args, rank, world):
    if rank != 0:
        return
    import oracle
    w = {"csr": gen.config("cfg1", args.seed, scale=16)}
    c = w["csr"]
    rr = gen.config("cfg2", args.seed, n=32_768)
    lj = gen.config("cfg3", args.seed, m=20)

    def step():
        inter = 0
        for red in (oracle.SUM, oracle.MAX):
            y, A, arg = oracle.csr_forward(c["rowptr"], c["col"], c["x"], c["w"], red)
            if red == oracle.SUM:
                oracle.csr_backward_sum(c["rowptr"], c["col"], c["x"], c["w"], c["gy"])
            else:
                oracle.csr_backward_max(c["rowptr"], c["col"], c["x"], c["w"], c["gy"], arg)
            inter += 2 * c["E"]
        oracle.degree_histogram(c["rowptr"], 4096)
        _, _, cnt = oracle.radius_forward(rr["pos"], rr["x"], rr["r"], rr["box"], rr["periodic"], oracle.MSG_GAUSS,
                                          p0=rr["sigma"], use_cells=True)
        oracle.radius_backward_gauss(rr["pos"], rr["x"], rr["gy"], rr["r"], rr["box"], rr["periodic"], rr["sigma"], use_cells=True)
        inter += 2 * int(cnt.sum())
        _, _, cnt = oracle.radius_forward(lj["pos"], None, lj["r"], lj["box"], lj["periodic"], oracle.MSG_LJ, 1.0, 1.0, use_cells=True)
        inter += int(cnt.sum())
        return inter

    for _ in range(min(args.warmup, 1)):
        step()
    t0 = time.time()
    inter = 0
    for _ in range(args.steps):
        inter += step()
    dt = time.time() - t0
    value = inter / dt
    sample = ("every row of the step on scaled-down replicas: R-MAT scale 16 (1,048,576 edges, F=64), "
              "32,768-point periodic Gaussian radius, 8,000-particle Lennard-Jones")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "bounded sample of: cfg1 CSR + cfg2 radius + cfg3 Lennard-Jones (" + sample + ")", "seed": args.seed},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_paper_shapes(args):
    """The paper's own workload shapes (Sections 7.1-7.3 and the fixed-topology study), timed the
    paper's way: warm, 4 warm-up calls, 10 timed calls, median.  Prints one JSON object."""
    import torch
    from paper_2609_24802_b200 import api as T
    dev = torch.device("cuda", 0)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    def median_ms(fn, warm=4, reps=10):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts), min(ts), max(ts)

    rows = []

    def csr_row(name, rowptr, col, n, F, paper):
        g = T.CsrRelation(rowptr, col, n)
        E = col.numel()
        x = torch.randn((n, F), device=dev)
        w = torch.rand(E, device=dev)
        out = torch.empty((n, F), device=dev)
        ws = torch.empty(T.tiga_csr_workspace_bytes(g, F, T.F32, T.SUM), dtype=torch.uint8, device=dev)
        med, lo, hi = median_ms(lambda: T.tiga_apply_csr(g, x, w, T.SUM, out=out, ws=ws))
        rows.append({"shape": name, "edges": E, "F": F, "ms_median": med, "ms_min": lo, "ms_max": hi,
                     "edges_per_s": E / (med * 1e-3), "paper": paper})

    for n in (8192, 32768, 131072):
        rp, col = gen.regular_random_csr(n, 32, args.seed)
        csr_row(f"stored CSR, degree 32, F=32, N={n}", to(rp), to(col), n, 32,
                "0.047-0.272 ms over the three sizes (RTX 5070 Ti)")
    rp, col = gen.regular_random_csr(32768, 32, args.seed)
    csr_row("stored CSR, degree 32, F=128, N=32768", to(rp), to(col), 32768, 128, "0.395 ms; Torch sparse 0.289 ms (RTX 5070 Ti)")
    rp, col = gen.hex_mesh_csr(96)
    csr_row("hex mesh L=96 (884,736 nodes, 22,508,920 edges), F=16", to(rp), to(col), 96 ** 3, 16, "23.00 ms, whole graph on one RTX 5070 Ti")
    offs = torch.tensor([1, 2, 3, 5, 8, 13, 21, 34, -1, -2, -3, -5, -8, -13, -21, -34], device=dev, dtype=torch.int64)
    for n in (625_000, 6_250_000, 62_500_000):
        rp = (torch.arange(n + 1, device=dev, dtype=torch.int64) * 16).to(torch.int64 if n * 16 >= 2**31 else torch.int32)
        col = torch.empty(n * 16, device=dev, dtype=torch.int32)
        step = 1 << 22
        for i0 in range(0, n, step):          # built on the device in slices (index arithmetic only)
            i1 = min(n, i0 + step)
            col[i0 * 16:i1 * 16] = ((torch.arange(i0, i1, device=dev, dtype=torch.int64)[:, None] + offs[None, :]) % n).to(torch.int32).reshape(-1)
        csr_row(f"periodic 16-neighbour CSR, F=32, {n * 16:,} edges, HBM resident", rp, col, n, 32,
                "1B edges: 414 s end to end with disk/host paging, CUDA kernels 1.60 s (RTX 5070 Ti)" if n == 62_500_000 else "figure only")
        del rp, col
        torch.cuda.empty_cache()
    for n in (8192, 32768, 131072):
        c = gen.config("cfg0", args.seed, n=n, nbrs=32.0, F=1)
        pos, x = to(c["pos"]), to(c["x"])
        out = torch.empty((n, 1), device=dev); cnt = torch.empty(n, dtype=torch.int32, device=dev)
        ws = torch.empty(T.tiga_radius_workspace_bytes(n, 1, c["r"], c["box"], c["periodic"]), dtype=torch.uint8, device=dev)
        med, lo, hi = median_ms(lambda: T.tiga_apply_radius(pos, x, c["r"], c["box"], c["periodic"], T.MSG_DIST, out=out, count=cnt, ws=ws))
        pairs = int(cnt.sum().item())
        rows.append({"shape": f"dynamic radius (rebuilt every call), distance-weighted scalar sum, N={n}", "pairs": pairs, "F": 1,
                     "ms_median": med, "ms_min": lo, "ms_max": hi, "interactions_per_s": pairs / (med * 1e-3),
                     "paper": "1.84 ms at N=131,072 (PyG 80.24 ms, chunked Torch 1870 ms; RTX 5070 Ti)" if n == 131072 else "figure only"})
    # differentiated edge network (Appendix A / supplementary study): 35,947 points on a synthetic closed
    # surface, cutoff 0.015, 8 node features, 4 outputs; forward includes the relation rebuild
    n = 35_947
    pos, x, gy = to(gen.surface_points(n, args.seed)), to(gen.normal_features(n, 8, args.seed, 31)), to(gen.normal_features(n, 4, args.seed, 32))
    ones, nonper = np.ones(3, np.float32), [0, 0, 0]
    for hidden, paper in ((8, "fwd 0.86 ms, loss+bwd 0.72 ms (Torch 0.64 / 2.07)"), (16, "example width, no timing printed"),
                          (32, "fwd 0.92 ms, loss+bwd 8.86 ms (Torch 0.94 / 2.42)")):
        P = [to(a) for a in gen.mlp_params(8, hidden, 4, args.seed)]
        out, cnt, ws = T.tiga_apply_radius_mlp(pos, x, 0.015, ones, nonper, *P, want_count=True)
        pairs = int(cnt.sum().item())
        fwd = median_ms(lambda: T.tiga_apply_radius_mlp(pos, x, 0.015, ones, nonper, *P, out=out, ws=ws))
        bwd = median_ms(lambda: T.tiga_apply_radius_mlp_backward(pos, x, gy, 0.015, ones, nonper, *P, ws=ws, reuse_plan=True))
        rows.append({"shape": f"edge network on a radius graph, 35,947 surface points, r=0.015, hidden {hidden}", "pairs": pairs,
                     "ms_median": fwd[0], "ms_min": fwd[1], "ms_max": fwd[2], "backward_ms_median": bwd[0],
                     "backward_ms_min": bwd[1], "backward_ms_max": bwd[2], "interactions_per_s": pairs / (fwd[0] * 1e-3),
                     "paper": paper + " on the Stanford Bunny vertices, 356,260 edges (RTX 5070 Ti)"})
    # online-softmax reducer: graph attention over the benchmark's stored relation and causal attention
    # as a stored triangular relation (the appendix' example shape, longer)
    c = gen.config("cfg1", args.seed)
    g = T.CsrRelation(to(c["rowptr"]), to(c["col"]), c["n"])
    q, k, v = (to(gen.normal_features(c["n"], 64, args.seed, 31 + i)) for i in range(3))
    out, lse, ws = T.tiga_apply_csr_attention(g, q, k, v, 0.125)
    med, lo, hi = median_ms(lambda: T.tiga_apply_csr_attention(g, q, k, v, 0.125, out=out, lse=lse, ws=ws))
    rows.append({"shape": "online-softmax reducer (graph attention), R-MAT scale 20, 16,777,216 edges, width 64", "edges": c["E"],
                 "F": 64, "ms_median": med, "ms_min": lo, "ms_max": hi, "edges_per_s": c["E"] / (med * 1e-3),
                 "gather_GBps": c["E"] * 512 / (med * 1e-3) / 1e9, "paper": "not measured in the paper"})
    del g, q, k, v, out, lse, ws
    for n in (4096, 16384):
        rp = torch.cat([torch.zeros(1, device=dev, dtype=torch.int64), torch.cumsum(torch.arange(1, n + 1, device=dev, dtype=torch.int64), 0)])
        e = torch.arange(int(rp[-1].item()), device=dev, dtype=torch.int64)
        col = (e - rp[torch.searchsorted(rp, e, right=True) - 1]).to(torch.int32)      # row i holds sources 0..i
        del e
        g = T.CsrRelation(rp, col, n)
        q, k, v = (torch.randn((n, 64), device=dev) for _ in range(3))
        out, lse, ws = T.tiga_apply_csr_attention(g, q, k, v, 0.125)
        med, lo, hi = median_ms(lambda: T.tiga_apply_csr_attention(g, q, k, v, 0.125, out=out, lse=lse, ws=ws))
        E = col.numel()
        rows.append({"shape": f"online-softmax reducer, causal attention as a stored triangular relation, {n} tokens, width 64", "edges": E,
                     "F": 64, "ms_median": med, "ms_min": lo, "ms_max": hi, "edges_per_s": E / (med * 1e-3),
                     "paper": "appendix example (65 tokens) is a correctness check; the paper's dense streaming path is not timed"})
        del g, q, k, v, out, lse, ws, rp, col
    # generated exact kNN, scalar neighbour sum, k = 16, relation rebuilt from the coordinates every call
    knn_paper = {1024: "0.147 ms (Torch 0.244, PyG 1.775)", 16384: "6.32 ms (Torch 29.92, PyG 17.50)",
                 131072: "172.37 ms (Torch 1908.43, PyG 393.21)"}
    for n in (1024, 4096, 16384, 32768, 65536, 131072, 1_000_000, 4_000_000):
        pos, x = to(gen.uniform_points(n, args.seed)), to(gen.normal_features(n, 1, args.seed, 31))
        out, nbr, d2, ws = T.tiga_apply_knn(pos, x, 16, ones)
        med, lo, hi = median_ms(lambda: T.tiga_apply_knn(pos, x, 16, ones, out=out, nbr=nbr, nbr_d2=d2, ws=ws))
        rows.append({"shape": f"generated exact kNN, k=16, scalar neighbour sum, N={n}", "pairs": 16 * n, "F": 1,
                     "ms_median": med, "ms_min": lo, "ms_max": hi, "interactions_per_s": 16 * n / (med * 1e-3),
                     "paper": (knn_paper.get(n, "figure only") + " (RTX 5070 Ti, all-pairs scan)") if n <= 131072 else "beyond the paper's sizes"})
        del pos, x, out, nbr, d2, ws
    c = gen.config("cfg2", args.seed, F=8)
    pos, x, gy = to(c["pos"]), to(c["x"]), to(gen.normal_features(c["n"], 4, args.seed, 33))
    P = [to(a) for a in gen.mlp_params(8, 16, 4, args.seed)]
    out, cnt, ws = T.tiga_apply_radius_mlp(pos, x, c["r"], c["box"], c["periodic"], *P, want_count=True)
    pairs = int(cnt.sum().item())
    fwd = median_ms(lambda: T.tiga_apply_radius_mlp(pos, x, c["r"], c["box"], c["periodic"], *P, out=out, ws=ws))
    bwd = median_ms(lambda: T.tiga_apply_radius_mlp_backward(pos, x, gy, c["r"], c["box"], c["periodic"], *P, ws=ws, reuse_plan=True))
    flop_f = 2.0 * (16 * 11 + 4 * 16) * pairs
    rows.append({"shape": "edge network, 1,000,000 periodic points, 32 neighbours, 8 features, hidden 16", "pairs": pairs,
                 "ms_median": fwd[0], "ms_min": fwd[1], "ms_max": fwd[2], "backward_ms_median": bwd[0],
                 "backward_ms_min": bwd[1], "backward_ms_max": bwd[2], "interactions_per_s": pairs / (fwd[0] * 1e-3),
                 "forward_tflops_fp32": flop_f / (fwd[0] * 1e-3) / 1e12, "paper": "not measured in the paper"})
    print(json.dumps({"case": "paper_shapes", "protocol": "warm, 4 warm-ups, 10 timed calls, median (min, max)", "rows": rows}))


def run_case(args):
    """One traversal on a reduced replica of its workload, a few launches, for profiler
    captures of a single kernel (`--case csr|radius_gauss|radius_lj --size S`)."""
    import torch
    from paper_2609_24802_b200 import api as T
    dev = torch.device("cuda", 0)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    ev0 = torch.cuda.Event(enable_timing=True); ev1 = torch.cuda.Event(enable_timing=True)
    if args.case == "csr":
        c = gen.config("cfg1", args.seed, scale=args.size or 18)
        g = T.CsrRelation(to(c["rowptr"]), to(c["col"]), c["n"])
        x, w, gy = to(c["x"]), to(c["w"]), to(c["gy"])
        def run():
            out, arg = T.tiga_apply_csr(g, x, w, T.SUM)
            T.tiga_apply_csr_backward(g, x, w, gy, T.SUM)
            om, am = T.tiga_apply_csr(g, x, w, T.MAX)
            T.tiga_apply_csr_backward(g, x, w, gy, T.MAX, argmax=am)
        units = c["E"]
    elif args.case == "csr_large":
        c = gen.config("cfg4", args.seed, scale=args.size or 26)
        g = T.CsrRelation(to(c["rowptr"]), to(c["col"]), c["n"])
        x = to(c["x"])
        out = torch.empty((c["n"], c["F"]), device=dev)
        ws = torch.empty(T.tiga_csr_workspace_bytes(g, c["F"], T.F16, T.SUM), dtype=torch.uint8, device=dev)
        def run():
            T.tiga_apply_csr(g, x, None, T.SUM, out=out, ws=ws)
        units = c["E"]
    elif args.case == "radius_gauss":
        c = gen.config("cfg2", args.seed, n=args.size or 300_000)
        pos, x, gy = to(c["pos"]), to(c["x"]), to(c["gy"])
        def run():
            out, cnt, ws = T.tiga_apply_radius(pos, x, c["r"], c["box"], c["periodic"], T.MSG_GAUSS, p0=c["sigma"])
            T.tiga_apply_radius_backward(pos, x, gy, c["r"], c["box"], c["periodic"], c["sigma"], ws=ws, reuse_plan=True)
        units = c["n"]
    elif args.case == "attention":
        c = gen.config("cfg1", args.seed, scale=args.size or 20)
        g = T.CsrRelation(to(c["rowptr"]), to(c["col"]), c["n"])
        q, k, v = (to(gen.normal_features(c["n"], 64, args.seed, 31 + i)) for i in range(3))
        out, lse, ws = T.tiga_apply_csr_attention(g, q, k, v, 0.125)
        def run():
            T.tiga_apply_csr_attention(g, q, k, v, 0.125, out=out, lse=lse, ws=ws)
        units = c["E"]
    elif args.case == "knn":
        n = args.size or 1_000_000
        pos, x = to(gen.uniform_points(n, args.seed)), to(gen.normal_features(n, 1, args.seed, 31))
        out, nbr, d2, ws = T.tiga_apply_knn(pos, x, 16, np.ones(3, np.float32))
        def run():
            T.tiga_apply_knn(pos, x, 16, np.ones(3, np.float32), out=out, nbr=nbr, nbr_d2=d2, ws=ws)
        units = n
    else:
        c = gen.config("cfg3", args.seed, m=args.size or 100)
        pos = to(c["pos"])
        cnt = torch.empty(c["n"], dtype=torch.int32, device=dev) if args.with_count else None
        def run():
            T.tiga_apply_radius(pos, None, c["r"], c["box"], c["periodic"], T.MSG_LJ, p0=1.0, p1=1.0, count=cnt)
        units = c["n"]
    for _ in range(max(args.warmup, 1)):
        run()
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(args.steps):
        run()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    rec = {"case": args.case, "units": units, "ms_per_step": ms, "units_per_s": units / (ms * 1e-3)}
    if args.case == "csr_large":
        # the HBM-stream test: the three bandwidth fractions against the measured copy bandwidth
        peaks = measured_peaks()
        hbm = peaks[0] * 1e9
        E, N = c["E"], c["n"]
        b_alg = E * (4 + 16) + N * (8 + 32)                       # col + one 16-byte source row per edge; rowptr + fp32 output row per row
        touched = int(torch.unique(g.col).numel()) if E <= (1 << 28) else None
        b_min = 8.0 * (N + 1) + 4.0 * E + 16.0 * (touched if touched is not None else 2.7e7) + 32.0 * N
        b_dram = 35.5e9 * E / float(1 << 30)                      # profiles/csr_large_cfg4_dram_traffic.md, per edge
        sink = torch.zeros(1, device=dev)
        for _ in range(2):
            T.tiga_probe_row_gather(x, g.col, sink)
        pa = torch.cuda.Event(enable_timing=True); pb = torch.cuda.Event(enable_timing=True)
        pa.record()
        for _ in range(3):
            T.tiga_probe_row_gather(x, g.col, sink)
        pb.record(); torch.cuda.synchronize()
        t_gather = pa.elapsed_time(pb) / 3
        rec.update({"gather_of_own_index_stream_ms": t_gather, "T_own_gather_over_T": t_gather / ms,
                    "gather_note": "tiga_probe_row_gather on the same col stream and feature table: the gathers alone, no row sums, no output",
                    "f_alg": b_alg / (ms * 1e-3) / hbm, "f_dram": b_dram / (ms * 1e-3) / hbm, "f_min": b_min / (ms * 1e-3) / hbm,
                    "bytes_alg": b_alg, "bytes_dram_ncu": b_dram, "bytes_min": b_min,
                    "bytes_dram_note": "ncu capture at full size scaled by edges: meaningful at scale 26 only (smaller feature tables fit L2)",
                    "touched_source_rows": touched if touched is not None else "2.7e7 (analytic, R-MAT scale 26)",
                    "peak_GBps": peaks[0], "peak_source": peaks[2] if len(peaks) > 2 else "measured"})
    print(json.dumps(rec))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=gen.DEFAULT_SEED)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", default=None, choices=["csr", "csr_large", "radius_gauss", "radius_lj", "knn", "attention", "paper_shapes"],
                    help="run one traversal on a reduced replica (for profiler captures) instead of the benchmark")
    ap.add_argument("--with-count", action="store_true", help="--case radius_lj: also ask for the neighbour counts")
    ap.add_argument("--size", type=int, default=0, help="--case size: R-MAT scale, number of points, or lattice side")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.case == "paper_shapes":
        run_paper_shapes(args)
    elif args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
