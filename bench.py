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
NOMINAL_HBM_GBS = 8000.0          # the nominal figure the targets were written against
TARGET = {"csr": 0.70, "radius": 0.50}

# (row, config, family).  One step runs every row once.
ROWS = [("csr_sum_fwd", "cfg1", "csr"), ("csr_sum_bwd", "cfg1", "csr"), ("csr_max_fwd", "cfg1", "csr"),
        ("csr_max_bwd", "cfg1", "csr"), ("csr_hist", "cfg1", None),
        ("radius_gauss_fwd", "cfg2", "radius"), ("radius_gauss_bwd", "cfg2", "radius"),
        ("radius_lj_fwd", "cfg3", "radius"),
        ("csr_large_fwd", "cfg4", "csr"), ("csr_large_hist", "cfg4", None),
        ("radius_tiny_fwd", "cfg0", None), ("radius_tiny_bwd", "cfg0", None)]


def make_workloads(seed, large=True):
    """Two input snapshots (seed, seed + 1) of every configuration; timed calls alternate between
    them.  The billion-edge relation is generated once; its two snapshots differ in the features."""
    t0 = time.time()
    snaps = []
    for s in (seed, seed + 1):
        snaps.append({"cfg0": gen.config("cfg0", s), "cfg1": gen.config("cfg1", s), "cfg2": gen.config("cfg2", s),
                      "cfg3": gen.config("cfg3", s)})
    if large:
        c4 = gen.config("cfg4", seed)
        snaps[0]["cfg4"] = c4
        alt = dict(c4)
        alt["x"] = gen.normal_features(c4["n"], c4["F"], seed + 1, 31, np.float16)
        snaps[1]["cfg4"] = alt
    return snaps, time.time() - t0


def input_hashes(snaps):
    out = {}
    for k, snap in enumerate(snaps):
        for name, c in snap.items():
            if name == "cfg4" and k == 1:
                out["cfg4/features_b"] = gen.sha256_of(c["x"])[:16]
                continue
            arrs = [c[a] for a in ("rowptr", "col", "w", "x", "gy", "pos") if c.get(a) is not None]
            out[f"{name}/{'ab'[k]}"] = gen.sha256_of(*arrs)[:16]
    return out


# DRAM traffic per unit measured with ncu on reduced replicas (profiles/*.md), used to scale
# `traffic` to a full launch: bytes per particle / point / edge of one launch of the row's kernels.
TRAFFIC_PER_UNIT = {
    "radius_lj_fwd": ("particle", 48.4),          # profiles/radius_lj_pairs_1M.md: 32.4 B measured + the 16-byte row that leaves L2 at full size
    "radius_gauss_fwd": ("point", 186.7),         # profiles/radius_traverse_gaussian_300k.md
    "radius_gauss_bwd": ("point", 364.6),
    "csr_sum_fwd": ("edge", 21.3),                # profiles/csr_kernels_rmat_scale18.md
    "csr_max_fwd": ("edge", 37.4),
    "csr_sum_bwd": ("edge", 45.4),
    "csr_max_bwd": ("edge", 51.9),
    "csr_large_fwd": ("edge", 33.1),              # profiles/csr_large_cfg4_dram_traffic.md (unplanned kernels)
}


def work_models(snap, counts, clock_mhz):
    """Algorithmic work per launch of every row.

    CSR: cache-oblivious gather model, bytes = E (col + w + one source row) + N (rowptr + one output
    row); backward adds the cotangent row, the read-modify-write of the source-gradient row and the
    edge gradient.  bytes_min: every touched byte once.  Radius: fp32 lane operations (FMA = 1), 7 per
    candidate pair of a 27-cell stencil plus F+3 (Gaussian forward), 3F+12 (Gaussian backward) or 14
    (Lennard-Jones) per accepted pair.
    """
    m = {}
    c = snap["cfg1"]
    E, N, F = c["E"], c["n"], c["F"]
    fb = 4 * F
    touched = counts["cfg1_touched"]
    m["csr_sum_fwd"] = dict(alg=E * (8 + fb) + N * (4 + fb), mn=4 * (N + 1) + 8 * E + fb * touched + fb * N, gather=E * fb, inter=E)
    m["csr_max_fwd"] = dict(alg=E * (8 + fb) + N * (4 + 2 * fb), mn=4 * (N + 1) + 8 * E + fb * touched + 2 * fb * N, gather=E * fb, inter=E)
    m["csr_sum_bwd"] = dict(alg=E * (8 + fb + 4 + 2 * fb) + N * (4 + fb) + N * fb,
                            mn=4 * (N + 1) + 8 * E + fb * touched + fb * N + 4 * E + fb * N, gather=2 * E * fb, inter=E)
    m["csr_max_bwd"] = dict(alg=N * F * (4 + 4 + 4 + 4 + 4 + 8 + 8), mn=N * F * 8 + 4 * E + fb * N, gather=None, inter=E)
    if "cfg4" in snap:
        c4 = snap["cfg4"]
        E4, N4 = c4["E"], c4["n"]
        m["csr_large_fwd"] = dict(alg=E4 * (4 + 16) + N4 * (8 + 32),
                                  mn=8 * (N4 + 1) + 4 * E4 + 16 * counts["cfg4_touched"] + 32 * N4, gather=None, inter=E4)
    alu_peak = 148 * 128 * clock_mhz * 1e6      # fp32 lane operations per second
    for row, cfg, per_acc in (("radius_gauss_fwd", "cfg2", None), ("radius_gauss_bwd", "cfg2", None), ("radius_lj_fwd", "cfg3", 14)):
        cc = snap[cfg]
        n = cc["n"]
        acc = counts[cfg + "_pairs"]
        cand = 27.0 * n * n / counts[cfg + "_ncell"]             # candidate pairs of a 27-cell stencil
        if per_acc is None:
            per_acc = cc["F"] + 3 if row.endswith("fwd") else 3 * cc["F"] + 12
        m[row] = dict(ops=7 * cand + per_acc * acc, inter=acc, alu_peak=alu_peak)
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


def _stats(ms_list):
    return {"ms": round(statistics.median(ms_list), 4), "ms_min": round(min(ms_list), 4), "ms_max": round(max(ms_list), 4)}


# ------------------------------------------------------------------------------ our arm
def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2609_24802_b200 import api as T
    from paper_2609_24802_b200 import bench_probe

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    hbm_gbs, sm_max, peak_kind = measured_peaks()
    large = not args.skip_large
    snaps, gen_seconds = make_workloads(args.seed + 2 * rank, large)
    hashes = input_hashes(snaps) if rank == 0 else {}

    def pin(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

    # pinned host copies (for the end-to-end leg) and device-resident inputs, per snapshot
    H, D = [], []
    for k, snap in enumerate(snaps):
        h = {}
        c0, c1, c2, c3 = snap["cfg0"], snap["cfg1"], snap["cfg2"], snap["cfg3"]
        h.update({"rowptr": pin(c1["rowptr"]), "col": pin(c1["col"]), "w": pin(c1["w"]), "x": pin(c1["x"]), "gy": pin(c1["gy"]),
                  "rpos": pin(c2["pos"]), "rx": pin(c2["x"]), "rgy": pin(c2["gy"]), "ljpos": pin(c3["pos"]),
                  "tpos": pin(c0["pos"]), "tx": pin(c0["x"]), "tgy": pin(c0["gy"])})
        if large:
            c4 = snap["cfg4"]
            if k == 0:
                h.update({"Lrowptr": pin(c4["rowptr"]), "Lcol": pin(c4["col"])})
            else:
                h.update({"Lrowptr": H[0]["Lrowptr"], "Lcol": H[0]["Lcol"]})
            h["Lx"] = pin(c4["x"])
        H.append(h)
        d = {}
        for name, v in h.items():
            if k == 1 and name in ("Lrowptr", "Lcol"):
                d[name] = D[0][name]
            else:
                d[name] = v.to(dev)
        D.append(d)
    c0, c1, c2, c3 = (snaps[0][k] for k in ("cfg0", "cfg1", "cfg2", "cfg3"))
    N, E, F = c1["n"], c1["E"], c1["F"]
    n2, F2 = c2["n"], c2["F"]
    n3 = c3["n"]
    n0, F0 = c0["n"], c0["F"]
    G = [T.CsrRelation(d["rowptr"], d["col"], N) for d in D]
    if large:
        c4 = snaps[0]["cfg4"]
        N4, E4, F4 = c4["n"], c4["E"], c4["F"]
        GL = T.CsrRelation(D[0]["Lrowptr"], D[0]["Lcol"], N4)

    out_sum = torch.empty((N, F), device=dev); out_max = torch.empty((N, F), device=dev)
    arg = torch.empty((N, F), dtype=torch.int32, device=dev)
    gx = torch.empty((N, F), device=dev); gw = torch.empty(E, device=dev)
    gxm = torch.empty((N, F), device=dev); gwm = torch.empty(E, device=dev)
    ws_csr = torch.empty(T.tiga_csr_workspace_bytes(G[0], F, T.F32, T.MAX), dtype=torch.uint8, device=dev)
    rout = torch.empty((n2, F2), device=dev); rcount = torch.empty(n2, dtype=torch.int32, device=dev)
    rgx = torch.empty((n2, F2), device=dev); rgp = torch.empty((n2, 3), device=dev)
    ws_rad = torch.empty(T.tiga_radius_workspace_bytes(n2, F2, c2["r"], c2["box"], c2["periodic"]), dtype=torch.uint8, device=dev)
    ljout = torch.empty((n3, 4), device=dev); ljcount = torch.empty(n3, dtype=torch.int32, device=dev)
    ws_lj = torch.empty(T.tiga_radius_workspace_bytes(n3, 4, c3["r"], c3["box"], c3["periodic"]), dtype=torch.uint8, device=dev)
    tout = torch.empty((n0, F0), device=dev); tcount = torch.empty(n0, dtype=torch.int32, device=dev)
    tgx = torch.empty((n0, F0), device=dev); tgp = torch.empty((n0, 3), device=dev)
    ws_tiny = torch.empty(T.tiga_radius_workspace_bytes(n0, F0, c0["r"], c0["box"], c0["periodic"]), dtype=torch.uint8, device=dev)
    plan = None
    plan_info = None
    if large:
        Lout = torch.empty((N4, F4), device=dev)
        ws_L = torch.empty(T.tiga_csr_workspace_bytes(GL, F4, T.F16, T.SUM), dtype=torch.uint8, device=dev)
        if hasattr(T, "tiga_csr_plan_build") and not args.no_plan:
            torch.cuda.synchronize()
            p0 = torch.cuda.Event(enable_timing=True); p1 = torch.cuda.Event(enable_timing=True)
            p0.record()
            plan = T.tiga_csr_plan_build(GL, row_bytes=2 * F4)
            p1.record(); torch.cuda.synchronize()
            ws_plan = torch.empty(T.tiga_csr_planned_workspace_bytes(plan, F4, T.F16, T.SUM), dtype=torch.uint8, device=dev)
            plan_info = {"build_ms": round(p0.elapsed_time(p1), 3), "plan_bytes": plan.nbytes, "build_scratch_bytes": plan.scratch_bytes,
                         "hot_sources": plan.n_hot, "min_hot_in_degree": plan.min_hot_degree,
                         "edges_with_a_hot_source": plan.hot_edges, "hot_table_bytes_per_call": plan.n_hot * 2 * F4,
                         "note": "one-time preprocessing that depends on (rowptr, col) only: the sources named by the most "
                                 "edges are numbered densely and the index stream is rewritten; every call copies their "
                                 "feature rows into one compact L2-resident table (inside the timed call) and then runs the "
                                 "unchanged row-major traversal; the build is not part of the timed call"}

    stream = torch.cuda.current_stream()

    def large_fwd(d):
        if plan is not None:
            T.tiga_apply_csr_planned(plan, d["Lx"], None, T.SUM, out=Lout, ws=ws_plan)
        else:
            T.tiga_apply_csr(GL, d["Lx"], None, T.SUM, out=Lout, ws=ws_L)

    # the step in its independent parts; mark(i) records the event that closes row i - 1
    def part_csr(k, mark):
        d, g = D[k], G[k]
        T.tiga_apply_csr(g, d["x"], d["w"], T.SUM, out=out_sum, ws=ws_csr); mark(1)
        T.tiga_apply_csr_backward(g, d["x"], d["w"], d["gy"], T.SUM, grad_x=gx, grad_w=gw); mark(2)
        T.tiga_apply_csr(g, d["x"], d["w"], T.MAX, out=out_max, argmax=arg, ws=ws_csr); mark(3)
        T.tiga_apply_csr_backward(g, d["x"], d["w"], d["gy"], T.MAX, argmax=arg, grad_x=gxm, grad_w=gwm); mark(4)
        hist, mx = T.tiga_csr_degree_histogram(g, 4096); mark(5)
        return hist

    def part_radius(k, mark):
        d = D[k]
        T.tiga_apply_radius(d["rpos"], d["rx"], c2["r"], c2["box"], c2["periodic"], T.MSG_GAUSS, p0=c2["sigma"],
                            out=rout, count=rcount, ws=ws_rad); mark(6)
        T.tiga_apply_radius_backward(d["rpos"], d["rx"], d["rgy"], c2["r"], c2["box"], c2["periodic"], c2["sigma"],
                                     ws=ws_rad, reuse_plan=True, grad_feat=rgx, grad_pos=rgp); mark(7)

    def part_lj(k, mark):
        # forces and energies only, as the row is defined; the pair count of the metric comes from one
        # counting call per snapshot before the timed region
        T.tiga_apply_radius(D[k]["ljpos"], None, c3["r"], c3["box"], c3["periodic"], T.MSG_LJ, p0=c3["eps"], p1=c3["s"],
                            out=ljout, ws=ws_lj); mark(8)

    def part_large(k, mark, planned=True):
        if not large:
            mark(9); mark(10)
            return None
        if planned:
            large_fwd(D[k])
        else:
            T.tiga_apply_csr(GL, D[k]["Lx"], None, T.SUM, out=Lout, ws=ws_L)
        mark(9)
        hist, mx = T.tiga_csr_degree_histogram(GL, 4096); mark(10)
        return hist

    def part_tiny(k, mark):
        d = D[k]
        T.tiga_apply_radius(d["tpos"], d["tx"], c0["r"], c0["box"], c0["periodic"], T.MSG_GAUSS, p0=c0["sigma"],
                            out=tout, count=tcount, ws=ws_tiny); mark(11)
        T.tiga_apply_radius_backward(d["tpos"], d["tx"], d["tgy"], c0["r"], c0["box"], c0["periodic"], c0["sigma"],
                                     ws=ws_tiny, reuse_plan=True, grad_feat=tgx, grad_pos=tgp); mark(12)

    def step(k, ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record(stream)
        mark(0)
        part_csr(k, mark)
        part_radius(k, mark)
        part_lj(k, mark)
        part_large(k, mark)
        part_tiny(k, mark)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # pair counts of both snapshots (outside the timed region)
    pairs = []
    for k in range(2):
        T.tiga_apply_radius(D[k]["ljpos"], None, c3["r"], c3["box"], c3["periodic"], T.MSG_LJ, p0=c3["eps"], p1=c3["s"],
                            out=ljout, count=ljcount, ws=ws_lj)
        step(k)
        torch.cuda.synchronize()
        pairs.append({"cfg0": int(tcount.sum().item()), "cfg2": int(rcount.sum().item()), "cfg3": int(ljcount.sum().item())})
    W = max(args.warmup, 4)
    for k in range(W):
        step(k % 2)
    sync_all()

    def inter_of(k):
        return 4 * E + 2 * pairs[k]["cfg2"] + pairs[k]["cfg3"] + (E4 if large else 0) + 2 * pairs[k]["cfg0"]

    # ---- timed region: device-resident inputs, K steps, snapshots alternate
    nrow = len(ROWS)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nrow + 1)] for _ in range(args.steps)]
    l0 = T.launch_count()
    sync_all()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(args.steps):
        step(k % 2, evs[k])
    t_end.record(stream)
    sync_all()
    sampler.stop_flag.set()
    launches = T.launch_count() - l0
    total_ms = t_start.elapsed_time(t_end)
    row_ms = [[evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)] for i in range(nrow)]
    inter_total = sum(inter_of(k % 2) for k in range(args.steps))
    clocks = sampler.summary()

    # ---- end-to-end leg: inputs start in pinned host memory, results end in pinned host memory
    res_h = {"out_sum": torch.empty((N, F)).pin_memory(), "gx": torch.empty((N, F)).pin_memory(),
             "gw": torch.empty(E).pin_memory(), "out_max": torch.empty((N, F)).pin_memory(),
             "gxm": torch.empty((N, F)).pin_memory(), "gwm": torch.empty(E).pin_memory(),
             "hist": torch.empty(4096, dtype=torch.int64).pin_memory(),
             "rout": torch.empty((n2, F2)).pin_memory(), "rgx": torch.empty((n2, F2)).pin_memory(),
             "rgp": torch.empty((n2, 3)).pin_memory(), "ljout": torch.empty((n3, 4)).pin_memory(),
             "tout": torch.empty((n0, F0)).pin_memory(), "tgx": torch.empty((n0, F0)).pin_memory(),
             "tgp": torch.empty((n0, 3)).pin_memory()}
    if large:
        res_h.update({"Lout": torch.empty((N4, F4)).pin_memory(), "Lhist": torch.empty(4096, dtype=torch.int64).pin_memory()})
    h2d = sum(v.numel() * v.element_size() for v in H[0].values())
    d2h = sum(v.numel() * v.element_size() for v in res_h.values())

    # Three streams: inputs go up on one, kernels run on the bench stream, results come down on a third,
    # so that the copies of one part overlap the kernels and the copies of the others (PCIe is full
    # duplex).  Events order every buffer: inputs are overwritten only after the kernels that read
    # them, outputs only after their copy to the host.  All of it lies inside the timed region.  The
    # billion-edge relation is uploaded in full every step and applied without any precomputed plan.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    nomark = lambda i: None
    parts = {
        "csr": (["rowptr", "col", "w", "x", "gy"], lambda k: part_csr(k, nomark),
                lambda hist: [("out_sum", out_sum), ("gx", gx), ("gw", gw), ("out_max", out_max), ("gxm", gxm), ("gwm", gwm), ("hist", hist)]),
        "radius": (["rpos", "rx", "rgy"], lambda k: part_radius(k, nomark), lambda _: [("rout", rout), ("rgx", rgx), ("rgp", rgp)]),
        "lj": (["ljpos"], lambda k: part_lj(k, nomark), lambda _: [("ljout", ljout)]),
        "tiny": (["tpos", "tx", "tgy"], lambda k: part_tiny(k, nomark), lambda _: [("tout", tout), ("tgx", tgx), ("tgp", tgp)]),
    }
    if large:
        parts["large"] = (["Lrowptr", "Lcol", "Lx"], lambda k: part_large(k, nomark, planned=False),
                          lambda hist: [("Lout", Lout), ("Lhist", hist)])
    computed = {k: None for k in parts}      # events of the previous step
    drained = {k: None for k in parts}

    def e2e_step(k):
        # uploads always land in the buffers of snapshot 0 (the kernels of this leg read those)
        for name, (inputs, compute, outputs) in parts.items():
            if computed[name] is not None:
                s_in.wait_event(computed[name])
            with torch.cuda.stream(s_in):
                for key in inputs:
                    D[0][key].copy_(H[k][key], non_blocking=True)
                up = torch.cuda.Event(); up.record(s_in)
            stream.wait_event(up)
            if drained[name] is not None:
                stream.wait_event(drained[name])
            hist = compute(0)
            done = torch.cuda.Event(); done.record(stream)
            computed[name] = done
            s_out.wait_event(done)
            with torch.cuda.stream(s_out):
                for key, src in outputs(hist):
                    res_h[key].copy_(src, non_blocking=True)
                    src.record_stream(s_out)
                dn = torch.cuda.Event(); dn.record(s_out)
            drained[name] = dn

    def e2e_join():
        for ev in drained.values():
            if ev is not None:
                stream.wait_event(ev)

    e2e_step(0)
    e2e_join()
    sync_all()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for k in range(args.steps):
        e2e_step(k % 2)
    e2e_join()
    e1.record(stream)
    sync_all()
    e2e_ms = e0.elapsed_time(e1)
    # the end-to-end leg left snapshot-dependent inputs of snapshot k in D[0]: put snapshot 0 back
    for key, v in H[0].items():
        D[0][key].copy_(v)
    torch.cuda.synchronize()

    total_ms, e2e_ms, inter_all = combine_ranks(dist, dev, total_ms, e2e_ms, inter_total)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = inter_all / (total_ms * 1e-3)
    clock_for_alu = clocks["sm_mhz"] or sm_max

    # ---- probes outside the timed step (rank 0): L2 gather ceiling, gathers of the own index streams,
    #      warm and flushed L2, the unplanned billion-edge forward
    def timed(fn, reps=10, before=None, warm=2):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(reps):
            if before is not None:
                before()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    d0, g0 = D[0], G[0]
    gen_t = torch.Generator(device=dev); gen_t.manual_seed(args.seed)
    table = torch.randn((60 * 2**20 // (4 * F), F), device=dev, generator=gen_t)              # 60 MiB of 256-byte rows: fits L2
    ridx = torch.randint(0, table.shape[0], (E,), device=dev, generator=gen_t, dtype=torch.int32)
    sink = torch.zeros(1, device=dev)
    t_l2 = timed(lambda: bench_probe.row_gather(table, ridx, sink))
    t_col = timed(lambda: bench_probe.row_gather(d0["x"], d0["col"], sink))                 # the workload's own index stream and table
    l2_peak = E * 4.0 * F / (t_l2 * 1e-3)
    flush_buf = torch.empty(512 * 2**20, dtype=torch.uint8, device=dev)
    fwd_call = lambda: T.tiga_apply_csr(g0, d0["x"], d0["w"], T.SUM, out=out_sum, ws=ws_csr)
    t_warm = timed(fwd_call)
    t_cold = timed(fwd_call, before=lambda: flush_buf.zero_())
    counts = {"cfg1_touched": int(torch.unique(d0["col"]).numel()),
              "cfg2_pairs": pairs[0]["cfg2"], "cfg3_pairs": pairs[0]["cfg3"],
              "cfg2_ncell": int(np.prod(T.tiga_radius_grid(n2, c2["r"], c2["box"], c2["periodic"])[0])),
              "cfg3_ncell": int(np.prod(T.tiga_radius_grid(n3, c3["r"], c3["box"], c3["periodic"])[0]))}
    del table, ridx, flush_buf
    large_extra = None
    if large:
        seen = torch.zeros(N4, dtype=torch.bool, device=dev)
        step_e = 1 << 27
        for e_lo in range(0, E4, step_e):
            seen[d0["Lcol"][e_lo:e_lo + step_e].long()] = True
        counts["cfg4_touched"] = int(seen.sum().item())
        del seen
        t_gather4 = timed(lambda: bench_probe.row_gather(d0["Lx"], d0["Lcol"], sink), reps=3, warm=1)
        t_unplanned = timed(lambda: T.tiga_apply_csr(GL, d0["Lx"], None, T.SUM, out=Lout, ws=ws_L), reps=5, warm=1)
        large_extra = {"gather_of_own_index_stream_ms": round(t_gather4, 4), "unplanned_forward_ms": round(t_unplanned, 4)}

    models = work_models(snaps[0], counts, clock_for_alu)
    units = {"particle": n3, "point": n2, "edge": E}
    row_report = {}
    for i, (name, cfg, family) in enumerate(ROWS):
        if cfg == "cfg4" and not large:
            continue
        st = _stats(row_ms[i])
        t = st["ms"] * 1e-3
        rep = dict(st, config=cfg)
        mdl = models.get(name)
        if mdl is not None and mdl["inter"]:
            rep["interactions_per_s"] = mdl["inter"] / t
        if name in TRAFFIC_PER_UNIT:
            kind, per = TRAFFIC_PER_UNIT[name]
            rep["traffic"] = per * (E4 if name == "csr_large_fwd" else units[kind])
        if mdl is not None and "alg" in mdl:
            # the three bandwidth fractions, against the measured copy bandwidth and the nominal figure
            bw = {"alg": mdl["alg"] / t, "min": mdl["mn"] / t}
            if rep.get("traffic") is not None and not (name == "csr_large_fwd" and plan is not None):
                bw["dram"] = rep["traffic"] / t
            for k, v in bw.items():
                rep["f_" + k] = v / (hbm_gbs * 1e9)
                rep["f_" + k + "_vs_8TBps"] = v / (NOMINAL_HBM_GBS * 1e9)
            rep.update(bytes_alg=mdl["alg"], bytes_min=mdl["mn"])
            if cfg == "cfg1":
                # 96 % of this relation's gathers are served by L2: HBM does not bound these rows; the
                # binding resource is L2 -> SM gather bandwidth, measured by the probe
                rep["bound"] = "l2_gather"
                rep["unit"] = "GB/s"
                rep["peak"] = l2_peak / 1e9
                if mdl["gather"] is not None:
                    rep["achieved"] = mdl["gather"] / t / 1e9
                    rep["frac"] = rep["achieved"] / rep["peak"]
                    rep["T_l2roof_over_T"] = rep["frac"]
                    rep["target"] = TARGET["csr"]
                if name in ("csr_sum_fwd", "csr_max_fwd"):
                    rep["T_own_gather_over_T"] = (t_col * 1e-3) / t
                rep["hbm_note"] = "f_alg above 1 only says that L2 serves the gathers; it is not an HBM fraction"
            else:
                rep.update(bound="hbm", unit="GB/s", peak=hbm_gbs, achieved=bw["alg"] / 1e9, frac=rep["f_alg"], target=TARGET["csr"])
                if large_extra:
                    rep.update(large_extra)
                    rep["T_own_gather_over_T"] = large_extra["gather_of_own_index_stream_ms"] / st["ms"]
                    rep["variant"] = "planned (hot sources served from a compact L2-resident table)" if plan is not None else "unplanned"
                    if plan_info:
                        rep["plan"] = plan_info
        elif mdl is not None:
            ach = mdl["ops"] / t
            rep.update(bound="alu", unit="Tlaneop/s", peak=mdl["alu_peak"] / 1e12, achieved=ach / 1e12, frac=ach / mdl["alu_peak"],
                       target=TARGET["radius"])
        else:
            rep["bound"] = "launch"
        row_report[name] = rep
    row_report["csr_sum_fwd"].update(ms_back_to_back_warm_l2=round(t_warm, 4), ms_l2_flushed_512MiB_write_between_calls=round(t_cold, 4),
                                     touched_source_rows=counts["cfg1_touched"],
                                     l2_gather_peak_note="row-gather probe: 16.8M uniform random 256-byte row gathers from a 60 MiB table",
                                     gather_of_own_index_stream_ms=round(t_col, 4))

    judged = [k for k, v in row_report.items() if v.get("frac") is not None and v.get("target")]
    worst = min(judged, key=lambda k: row_report[k]["frac"] / row_report[k]["target"])
    dom = max(row_report, key=lambda k: row_report[k]["ms"])

    def roof(name):
        r = row_report[name]
        return {"kernel": name, "bound": r["bound"], "achieved": r.get("achieved"), "peak": r.get("peak"), "unit": r.get("unit"),
                "frac": r.get("frac"), "target": r.get("target"), "traffic": r.get("traffic"),
                "traffic_note": "ncu dram bytes of this row's kernels on a reduced replica, scaled by units processed (profiles/)",
                "peak_source": {"hbm": peak_kind + " hbm copy", "alu": peak_kind + " 148 SM x 128 lanes x sampled SM clock",
                                "l2_gather": "measured in this run by the row-gather probe"}.get(r["bound"], "")}

    t_of = lambda name: row_report[name]["ms"] * 1e-3
    fwd = {"csr_sum": E / t_of("csr_sum_fwd"), "csr_max": E / t_of("csr_max_fwd"),
           "radius_gauss": pairs[0]["cfg2"] / t_of("radius_gauss_fwd"), "radius_lj": pairs[0]["cfg3"] / t_of("radius_lj_fwd"),
           "radius_tiny": pairs[0]["cfg0"] / t_of("radius_tiny_fwd")}
    fwd_bwd = {"csr_sum": E / (t_of("csr_sum_fwd") + t_of("csr_sum_bwd")), "csr_max": E / (t_of("csr_max_fwd") + t_of("csr_max_bwd")),
               "radius_gauss": pairs[0]["cfg2"] / (t_of("radius_gauss_fwd") + t_of("radius_gauss_bwd")),
               "radius_tiny": pairs[0]["cfg0"] / (t_of("radius_tiny_fwd") + t_of("radius_tiny_bwd"))}
    if large:
        fwd["csr_large"] = E4 / t_of("csr_large_fwd")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD if large else WORKLOAD.replace(" + cfg4 CSR R-MAT scale 26 E=2^30 int64 rowptr F=8 fp16 (sum fwd, degree histogram)", ""),
                   "seed": args.seed,
                   "protocol": f"{W} warm-up steps, {args.steps} timed steps, inputs alternate between two snapshots (seed, seed+1; "
                               "the billion-edge relation keeps its graph and alternates its feature table); "
                               "per-row times are median (min, max) over the timed steps, CUDA events on the launching stream",
                   "l2": "inputs larger than L2 (644 MB of CSR inputs per snapshot, 5.8 GB for cfg4); consecutive steps use different snapshots",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "interactions_per_step": [inter_of(0), inter_of(1)], "pairs": pairs,
                   "lj_pairs_note": "counted by one call with neighbour counts before the timed region; the timed Lennard-Jones call returns forces and energies only",
                   "input_sha256_16": hashes, "input_generation_seconds": round(gen_seconds, 1)},
        "fwd_interactions_per_s": fwd, "fwd_bwd_interactions_per_s": fwd_bwd, "rows": row_report,
        "roofline": roof(worst), "roofline_note": "the row furthest below its target (frac / target smallest)",
        "roofline_longest_row": roof(dom),
        "e2e": {"value": inter_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "every input copied from pinned host memory and every result copied back inside the timed region, "
                        "copies and kernels pipelined over three streams; the billion-edge forward runs unplanned here"},
        "gpu_launches": launches, "gpu_launches_note": "counted inside the library (tiga_kernel_launches) around the timed region",
        "clocks": clocks,
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(snaps[0], large)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ CPU oracle arms
def cpu_baseline(snap, large=True):
    """The fp64 oracle, as it stands, on the step's workloads: one pass of every row."""
    import oracle
    legs = {}
    c = snap["cfg1"]
    t0 = time.time()
    _, _, arg = oracle.csr_forward(c["rowptr"], c["col"], c["x"], c["w"], oracle.MAX)
    oracle.csr_forward(c["rowptr"], c["col"], c["x"], c["w"], oracle.SUM)
    oracle.csr_backward_sum(c["rowptr"], c["col"], c["x"], c["w"], c["gy"])
    oracle.csr_backward_max(c["rowptr"], c["col"], c["x"], c["w"], c["gy"], arg)
    oracle.degree_histogram(c["rowptr"], 4096)
    legs["cfg1 CSR sum and max fwd + bwd, histogram"] = (4 * c["E"], time.time() - t0)
    rr = snap["cfg2"]
    t0 = time.time()
    _, _, cnt = oracle.radius_forward(rr["pos"], rr["x"], rr["r"], rr["box"], rr["periodic"], oracle.MSG_GAUSS,
                                      p0=rr["sigma"], use_cells=True)
    oracle.radius_backward_gauss(rr["pos"], rr["x"], rr["gy"], rr["r"], rr["box"], rr["periodic"], rr["sigma"], use_cells=True)
    legs["cfg2 radius Gaussian fwd + bwd (oracle's cell directory)"] = (2 * int(cnt.sum()), time.time() - t0)
    lj = snap["cfg3"]
    t0 = time.time()
    _, _, cnt3 = oracle.radius_forward(lj["pos"], None, lj["r"], lj["box"], lj["periodic"], oracle.MSG_LJ, 1.0, 1.0, use_cells=True)
    legs["cfg3 Lennard-Jones (oracle's cell directory)"] = (int(cnt3.sum()), time.time() - t0)
    if large:
        c4 = snap["cfg4"]
        t0 = time.time()
        oracle.csr_forward(c4["rowptr"], c4["col"], c4["x"], None, oracle.SUM)
        oracle.degree_histogram(c4["rowptr"], 4096)
        legs["cfg4 CSR sum fwd (straight loop, one pass), histogram"] = (c4["E"], time.time() - t0)
    t = snap["cfg0"]
    t0 = time.time()
    _, _, cnt0 = oracle.radius_forward(t["pos"], t["x"], t["r"], t["box"], t["periodic"], oracle.MSG_GAUSS, p0=t["sigma"])
    oracle.radius_backward_gauss(t["pos"], t["x"], t["gy"], t["r"], t["box"], t["periodic"], t["sigma"])
    legs["cfg0 radius Gaussian fwd + bwd (all pairs, brute force)"] = (2 * int(cnt0.sum()), time.time() - t0)
    inter = sum(v[0] for v in legs.values())
    secs = sum(v[1] for v in legs.values())
    return {"value": inter / secs, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "the whole step once (" + "; ".join(f"{k}: {v[0]} interactions in {v[1]:.1f} s" for k, v in legs.items()) + ")",
            "legs": {k: {"interactions": v[0], "seconds": round(v[1], 2), "interactions_per_s": v[0] / v[1]} for k, v in legs.items()}}


WORKLOAD = ("cfg1 CSR R-MAT scale 20 E=16,777,216 F=64 fp32 (sum fwd+bwd, max fwd+bwd, degree histogram) "
            "+ cfg2 radius N=1,000,000 periodic F=32 Gaussian (bin+fwd, bwd) "
            "+ cfg3 Lennard-Jones N=4,096,000 (bin+fwd)"
            " + cfg4 CSR R-MAT scale 26 E=2^30 int64 rowptr F=8 fp16 (sum fwd, degree histogram)"
            " + cfg0 radius N=4096 F=16 Gaussian (bin+fwd, bwd)")


def run_reference(args, rank, world):
    """The oracle, as it stands, on the host cores: every row of the step on a bounded sample."""
    if rank != 0:
        return
    import oracle
    c = gen.config("cfg1", args.seed, scale=16)
    rr = gen.config("cfg2", args.seed, n=32_768)
    lj = gen.config("cfg3", args.seed, m=20)
    c4 = gen.config("cfg4", args.seed, scale=18)
    t0c = gen.config("cfg0", args.seed)

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
        oracle.csr_forward(c4["rowptr"], c4["col"], c4["x"], None, oracle.SUM)
        oracle.degree_histogram(c4["rowptr"], 4096)
        inter += c4["E"]
        _, _, cnt = oracle.radius_forward(t0c["pos"], t0c["x"], t0c["r"], t0c["box"], t0c["periodic"], oracle.MSG_GAUSS, p0=t0c["sigma"])
        oracle.radius_backward_gauss(t0c["pos"], t0c["x"], t0c["gy"], t0c["r"], t0c["box"], t0c["periodic"], t0c["sigma"])
        inter += 2 * int(cnt.sum())
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
              "32,768-point periodic Gaussian radius, 8,000-particle Lennard-Jones, R-MAT scale 18 (4,194,304 edges, F=8 fp16), "
              "the 4096-point radius case in full")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample, "seed": args.seed},
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
    from paper_2609_24802_b200 import bench_probe
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
        plan = None
        if args.planned:
            # hot table scaled with the feature table: one sixteenth of the sources (64 MiB of 1 GiB at full size)
            plan = T.tiga_csr_plan_build(g, max_hot_rows=c["n"] // 16)
            wsp = torch.empty(T.tiga_csr_planned_workspace_bytes(plan, c["F"], T.F16, T.SUM), dtype=torch.uint8, device=dev)
        def run():
            if plan is not None:
                T.tiga_apply_csr_planned(plan, x, None, T.SUM, out=out, ws=wsp)
            else:
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
        # profiles/csr_large_cfg4_dram_traffic.md: bytes per edge of the unplanned design (once measured at
        # full size) or of the planned scale-24 replica (a lower bound at full size)
        b_dram = (15.7 if args.planned else 33.1) * E
        sink = torch.zeros(1, device=dev)
        for _ in range(2):
            bench_probe.row_gather(x, g.col, sink)
        pa = torch.cuda.Event(enable_timing=True); pb = torch.cuda.Event(enable_timing=True)
        pa.record()
        for _ in range(3):
            bench_probe.row_gather(x, g.col, sink)
        pb.record(); torch.cuda.synchronize()
        t_gather = pa.elapsed_time(pb) / 3
        rec.update({"gather_of_own_index_stream_ms": t_gather, "T_own_gather_over_T": t_gather / ms,
                    "gather_note": "row-gather probe on the same col stream and feature table: the gathers alone, no row sums, no output",
                    "f_alg": b_alg / (ms * 1e-3) / hbm, "f_dram": b_dram / (ms * 1e-3) / hbm, "f_min": b_min / (ms * 1e-3) / hbm,
                    "bytes_alg": b_alg, "bytes_dram_ncu": b_dram, "bytes_min": b_min,
                    "bytes_dram_note": ("planned: ncu capture of the scale-24 replica scaled by edges, a lower bound at scale 26" if args.planned else
                                        "unplanned: per-edge DRAM bytes of the full-size relation; smaller feature tables fit L2 and move less"),
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
    ap.add_argument("--skip-large", action="store_true", help="leave the billion-edge relation (cfg4) out of the step")
    ap.add_argument("--no-plan", action="store_true", help="apply the billion-edge relation without its source-block plan")
    ap.add_argument("--case", default=None, choices=["csr", "csr_large", "radius_gauss", "radius_lj", "knn", "attention", "paper_shapes"],
                    help="run one traversal on a reduced replica (for profiler captures) instead of the benchmark")
    ap.add_argument("--with-count", action="store_true", help="--case radius_lj: also ask for the neighbour counts")
    ap.add_argument("--planned", action="store_true", help="--case csr_large: apply through the hot-source plan")
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
