#!/usr/bin/env python
"""Benchmark of the GRF-masked linear-attention path: one step = sample the graph random features
(walks, merge, CSR, regrouping) and evaluate the masked attention for one batch of synthetic inputs.
Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload pc32768] [--route sz|mhat|asym]
                    [--frozen] [--impl ours|reference]
    python bench.py --suite        every workload, the unsorted point cloud, the scaling sweep and the operation
                                   counts of Sec. 4: a summary (.md) and one JSON line per run (.jsonl) in --suite-dir

Routes: sz = Alg. 1 through the per-node states S_l, z_l (Eq. 12; the headline); mhat = Eqs. 1-2 over the
materialised mask Phi Psi^T; asym = Alg. 2 (asymmetric features, Psi = I).

With N > 1 (launched by torch.distributed.run) every rank runs the same-sized, independently seeded batch
on its own GPU (the problems are independent: no data-path collective); the value is the sum of all
ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "grf_masked_linear_attention_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
CSRC = os.path.join(ROOT, "paper_2410_03462_b200", "csrc")
COUNTERS_FILE = os.path.join(ROOT, "profiles", "ncu_counters.md")
# Delivery of randomly addressed 4 KB bulk copies into shared memory with two issuing warps per SM (the gather
# kernel's configuration), measured once with a stand-alone copy loop on this GPU type: the resource that bounds
# the gather of state tiles.  Plain 16-byte loads of an L2-resident region reach 19.5 TB/s.
SMEM_FILL_PEAK_GBS = 6800.0


def make_workload(name: str):
    from workloads import configs
    if name.startswith("sweep"):
        return configs.sweep(int(name[5:]))
    if name == "pc32768-unsorted":
        return configs.point_cloud_32768(morton=False)
    return configs.BY_NAME[name]()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_PEAKS["hbm_gbs"], "bf16_tflops": FALLBACK_PEAKS["bf16_tflops"],
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def source_hash(files) -> str:
    """Hash of the kernel sources a profile entry was taken from (first 16 hex digits of SHA-256)."""
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def load_counters():
    """The tracked table of profiler counters, one row per kernel class:
    | class | sources | source hash | workload | heads captured | dram bytes per launch at capture | issue % | tensor % | lsu % |
    A row whose hash no longer matches the sources is stale: its figures are reported as null."""
    out = {}
    if not os.path.exists(COUNTERS_FILE):
        return out
    with open(COUNTERS_FILE) as fh:
        for line in fh:
            cells = [c.strip() for c in line.strip().strip("|").split("|")]
            if len(cells) < 9 or cells[0] in ("class", "") or set(cells[0]) <= set("-: "):
                continue
            try:
                files = cells[1].split()
                out[cells[0]] = {"sources": files, "hash": cells[2], "workload": cells[3], "heads": int(cells[4]),
                                 "dram_bytes": float(cells[5]), "issue_pct": float(cells[6]), "tensor_pct": float(cells[7]),
                                 "lsu_pct": float(cells[8]), "stale": source_hash(files) != cells[2]}
            except (ValueError, OSError):
                continue
    return out


class ClockSampler:
    """nvidia-smi clock/throttle samples every 10 ms while the timed region runs (read-only queries)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={device_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "10"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and throttle reasons over the samples taken between the two wall-clock times
        (all samples if none falls inside)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        rows = []
        for line in self.tmp:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), parts[5:9]))
            except ValueError:
                continue
        self.tmp.close()
        os.unlink(self.tmp.name)
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        use = inside or rows
        reasons = set()
        for _, _, _, flags in use:
            for name, flag in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), flags):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if use:
            out.update(sm_mhz=statistics.median(r[1] for r in use), sm_max_mhz=max(r[2] for r in use),
                       reasons=sorted(reasons), samples=len(use), window="timed region" if inside else "whole run")
        return out


def algorithmic_bytes(w, N, nnz_phi, nnz_psi, E):
    """Bytes each kernel class must move per step if every operand crosses HBM exactly once."""
    es = 2 if w.dtype == "bf16" else 4
    G, m, d = w.G, w.m, w.d
    S = G * N * m * d * es
    z = G * N * m * 4
    zb = G * N * m * 2 if w.dtype == "bf16" else 0          # bf16 copy of z in the records
    csr = lambda nnz: nnz * 8 + (N + 1) * 4
    return {
        # graph read once; merged rows written once
        "walk_merge": E * 8 + (N + 1) * 4 + (nnz_phi + nnz_psi) * 8 + 2 * N * 4,
        "scan": 2 * N * 4 * 3,
        "compact": 2 * (nnz_phi + nnz_psi) * 8,
        "regroup": 3 * csr(nnz_psi),
        # phi(K), V, Psi^T read once; S and z written once
        "build_states": G * N * (m + d) * es + csr(nnz_psi) + S + z + zb,
        # S, z, phi(Q), Phi read once; out written once
        "gather_contract": S + z + G * N * m * es + csr(nnz_phi) + G * N * d * es,
        # z and Phi read once, denominators written once
        "row_denominators": (zb if zb else z) + csr(nnz_phi) + G * N * m * es + G * N * 4,
        # Phi read twice (union lists, coefficient table)
        "block_plan": 2 * csr(nnz_phi),
    }


def binding_report(w, N, nnz_phi, nnz_psi, ktimes, steps, pk, counters, plan_entries, mask_entries):
    """For each big kernel, the rates of the resources that can bind it (from counts of this run and the CUDA-event
    time of the kernel) and, where the tracked profile of the same sources exists, the profiler's busy fractions.
    `binds` names the resource with the largest fraction of its peak."""
    es = 2 if w.dtype == "bf16" else 4
    G, m, d = w.G, w.m, w.d
    rep = {}

    def per_launch_s(name):
        ms, n = ktimes.get(name, (0.0, 0))
        return (ms / n) * 1e-3 if n else None

    def prof(name):
        c = counters.get(name)
        if not c or c["stale"]:
            return {"profile": "none for these sources" if not c else "stale (sources changed since the capture)"}
        return {"issue_slots_busy_pct": c["issue_pct"], "tensor_pipe_busy_pct": c["tensor_pct"],
                "lsu_pipe_busy_pct": c["lsu_pct"], "profile": f"{c['workload']}, {c['heads']} heads"}

    def finish(name, r, fracs):
        r["binds"] = max(fracs, key=fracs.get)
        r["fraction_of_binding_peak"] = fracs[r["binds"]]
        r.update(prof(name))
        rep[name] = r

    t = per_launch_s("gather_contract")
    if t and plan_entries and w.dtype == "bf16":
        issued = plan_entries * G * 2.0 * 128 * m * d / t / 1e12
        useful = 2.0 * nnz_phi * m * d * G / t / 1e12
        fill = plan_entries * G * m * d * es / t / 1e9
        hbm = (G * N * m * d * es) / t / 1e9
        finish("gather_contract", {
            "tensor_issued_tflops": issued, "tensor_useful_tflops": useful, "tensor_peak_tflops": pk["bf16_tflops"],
            "smem_fill_gbs": fill, "smem_fill_peak_gbs": SMEM_FILL_PEAK_GBS, "hbm_algorithmic_gbs": hbm},
            {"tensor_issue": issued / pk["bf16_tflops"], "smem_fill": fill / SMEM_FILL_PEAK_GBS, "hbm": hbm / pk["hbm_gbs"]})
    t = per_launch_s("build_states")
    if t and w.dtype == "bf16":
        gathered = (nnz_psi * G * (m + d) * es + G * N * (m * d * es + m * 6)) / t / 1e9
        issued = 2.0 * 128 * m * (nnz_psi + 8 * N) * G / t / 1e12       # keys padded to steps of 16 (8 on average)
        hbm = G * N * (m * d * es + m * 6) / t / 1e9
        finish("build_states", {
            "delivered_gbs": gathered, "delivery_peak_gbs": SMEM_FILL_PEAK_GBS, "tensor_issued_tflops": issued,
            "tensor_peak_tflops": pk["bf16_tflops"], "hbm_algorithmic_gbs": hbm},
            {"row_delivery": gathered / SMEM_FILL_PEAK_GBS, "tensor_issue": issued / pk["bf16_tflops"], "hbm": hbm / pk["hbm_gbs"]})
    t = per_launch_s("walk_merge")
    if t:
        keep = 1.0 - w.p_halt
        visits = (1.0 - keep ** (w.max_len + 1)) / w.p_halt        # expected nodes visited per walk (no dead ends)
        walks = 2.0 * N * w.n_walks
        c = counters.get("walk_merge")
        issue = (c["issue_pct"] / 100.0) if c and not c["stale"] else None
        r = {"walks_per_s": walks / t, "expected_hops_per_s": walks * (visits - 1.0) / t,
             "hbm_algorithmic_gbs": (8 * (nnz_phi + nnz_psi)) / t / 1e9}
        fr = {"hbm": r["hbm_algorithmic_gbs"] / pk["hbm_gbs"]}
        if issue is not None:
            fr["integer_issue"] = issue
        finish("walk_merge", r, fr)
    t = per_launch_s("mhat_attention")
    if t and mask_entries:
        issued = mask_entries * G * 2.0 * 128 * (m + d) / t / 1e12
        masked = mask_entries * 128.0 * G / t / 1e9                 # score entries multiplied by the mask per second
        hbm = (mask_entries * 260 + G * N * (2 * m + 2 * d) * es) / t / 1e9
        finish("mhat_attention", {
            "tensor_issued_tflops": issued, "tensor_peak_tflops": pk["bf16_tflops"], "masked_scores_g_per_s": masked,
            "hbm_algorithmic_gbs": hbm},
            {"tensor_issue": issued / pk["bf16_tflops"], "hbm": hbm / pk["hbm_gbs"]})
    return rep


def rank_seed(base: int, rank: int) -> int:
    """Every rank draws its own batch: same shapes, different values."""
    return base + rank


def aggregate_over_ranks(local_ms: float, tokens_per_rank_step: int, steps: int, world: int, reduce_max):
    """Whole-job throughput: all ranks' tokens over the slowest rank's device time."""
    total_ms = reduce_max(local_ms)
    return total_ms, tokens_per_rank_step * world * steps / (total_ms * 1e-3)


DTYPE_NOTE = {
    "sz": "bf16 storage, fp32 accumulation; tensor-core path multiplies bf16(Phi_il)*phi(q) and bf16(Psi_jl)*phi(k) rounded to bf16",
    "mhat": "bf16 storage, fp32 scores and mask sums; the mask and the masked scores are rounded to bf16",
    "asym": "bf16 storage, fp32 accumulation",
}


def measure(args, workload_name, route, with_cpu_baseline, with_e2e, frozen=False, steps=None, warmup=None,
            remodulate=False):
    """remodulate: the walks are sampled once and kept; every step gives them new coefficients (Alg. 1 with learnable
    f: grf_remodulate), prepares the feature object again and runs the attention."""
    import torch
    import torch.distributed as dist

    from paper_2410_03462_b200 import api, binding as B
    from workloads import configs, tensors

    steps = steps or args.steps
    warmup = warmup or args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    w = make_workload(workload_name)
    if args.heads > 0:
        w.heads = args.heads
        w.name += f"-heads{args.heads}"
    g = w.graph()
    N, E = g.N, g.E
    asym, mhat = route == "asym", route == "mhat"
    if asym:      # Alg. 2: f_phi = alpha, f_psi = delta_0 (no key-side walks contribute, Psi = I)
        f = w.alpha.astype(np.float32)
        f_psi = np.zeros(w.max_len + 1, np.float32); f_psi[0] = 1.0
    else:
        f = B.grf_deconvolve(w.alpha).astype(np.float32)
        f_psi = None
    ctx = api.Context(local)
    dg = api.DeviceGraph(g, local)
    # every rank has its own batch of the same shape (weak scaling over independent problems)
    q, k, v = tensors.qkv(w.G, N, w.m, w.d, w.dtype, rank_seed(configs.QKV_SEED, rank))
    if asym and args.softmax:     # keep the exponents moderate
        q, k = (q.float() * 0.25).to(q.dtype), (k.float() * 0.25).to(k.dtype)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    dt = B.dtype_code(qd)
    ws = None
    ws_bytes = 0
    if route == "sz":
        ws_bytes = B.grf_attn_workspace_bytes(w.G, N, w.m, w.d, dt)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    out = torch.empty_like(vd)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    feat = api.Features(ctx, None)

    def sample(seed):
        if remodulate and feat.handle is not None:
            # same walks, new coefficients (a small change of every f_t that differs from step to step)
            fi = (f * np.float32(1.0 - 0.001 * (seed % 7))).astype(np.float32)
            B.grf_remodulate(ctx.handle, feat.handle, w.max_len, fi, None if f_psi is None else f_psi)
            return
        feat.handle = B.grf_sample(ctx.handle, N, dg.rowptr, dg.col, dg.w, seed, w.n_walks, w.p_halt, w.max_len, f, f_psi,
                                   feat.handle)

    def prepare():        # what a feature object needs once before the attention can use it
        if mhat:
            B.grf_features_materialise(ctx.handle, feat.handle)

    def attention():
        if mhat:
            B.grf_masked_attn_mhat(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt, qd, kd, vd, out, None)
        elif asym:
            B.grf_masked_attn_asym(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt,
                                   B.GRF_KERNEL_SOFTMAX if args.softmax else B.GRF_KERNEL_LINEAR, qd, kd, vd, out, None)
        else:
            B.grf_masked_linear_attn(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt, qd, kd, vd, out, None, ws, ws_bytes)

    def step(seed):
        if not frozen:
            sample(seed)
            prepare()
        attention()

    sampler = ClockSampler(local) if rank == 0 else None
    B.grf_ctx_enable_timing(ctx.handle, True)      # per-kernel events exist before the timed region starts
    if remodulate:                                  # the walks themselves are kept with the features
        B.grf_ctx_keep_walks(ctx.handle, True)
        sample(configs.WALK_SEED)
        B.grf_ctx_keep_walks(ctx.handle, False)
        prepare()
    if frozen:                                      # walks "pre-computed and frozen" (Sec. 4): outside the step
        sample(configs.WALK_SEED)
        prepare()
    for i in range(warmup):
        step(configs.WALK_SEED + i)
    torch.cuda.synchronize()
    B.grf_ctx_kernel_times(ctx.handle)             # discard the warm-up record

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K steps, each bracketed by CUDA events on the stream the kernels run on;
    # L2 is flushed between steps, outside the events
    launches0 = ctx.launches
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    ev_mid = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    t_wall0 = time.perf_counter()
    t_epoch0 = time.time()
    for i in range(steps):
        flush.zero_()
        evs[i][0].record()
        if not frozen:
            sample(configs.WALK_SEED + 1000 + i)
        ev_mid[i].record()
        if not frozen:
            prepare()
        attention()
        evs[i][1].record()
    barrier()
    wall = time.perf_counter() - t_wall0
    t_epoch1 = time.time()
    launches = ctx.launches - launches0
    step_ms = [a.elapsed_time(b) for a, b in evs]
    sample_ms = [a[0].elapsed_time(mid) for a, mid in zip(evs, ev_mid)]
    attn_ms = [mid.elapsed_time(a[1]) for a, mid in zip(evs, ev_mid)]
    total_ms = sum(step_ms)
    ktimes = B.grf_ctx_kernel_times(ctx.handle)
    B.grf_ctx_enable_timing(ctx.handle, False)
    nnz_phi, nnz_psi = feat.shape(0)[2], feat.shape(1)[2]
    plan_entries = mask_entries = None
    if route == "sz" and w.dtype == "bf16":
        try:
            plan_entries = B.grf_plan_stats(ctx.handle, feat.handle)[1]
        except B.GrfError:
            plan_entries = None                     # no plan: the plain-ALU gather ran
    if mhat:
        mask_entries = B.grf_mask_stats(feat.handle)[1]

    # ---- end to end through the host-buffer entry point (pinned host memory; copies inside the timing)
    e2e = None
    if with_e2e and route in ("sz", "mhat") and not frozen and not remodulate:
        B.grf_ctx_prefer_mask_route(ctx.handle, mhat)
        qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
        oh = torch.empty_like(v).pin_memory()
        rp_h = torch.from_numpy(g.rowptr).pin_memory(); c_h = torch.from_numpy(g.col).pin_memory()
        w_h = torch.from_numpy(g.w).pin_memory()
        e2e_steps = max(2, min(steps, 5))

        def host_step(i):
            B.grf_step_host(ctx.handle, N, rp_h, c_h, w_h, configs.WALK_SEED + 2000 + i, w.n_walks, w.p_halt, w.max_len,
                            f, None, w.G, w.m, w.d, dt, qh, kh, vh, oh)

        host_step(0)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            host_step(1 + i)
        e1.record()
        barrier()
        e2e = {"ms": e0.elapsed_time(e1) / e2e_steps,
               "h2d": (rp_h.numel() + c_h.numel() + w_h.numel()) * 4 + sum(t.numel() * t.element_size() for t in (qh, kh, vh)),
               "d2h": oh.numel() * oh.element_size()}

    clocks = sampler.stop(t_epoch0, t_epoch1) if sampler else None

    # ---- max over ranks
    def rmax(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    total_ms, value = aggregate_over_ranks(total_ms, w.batch * N, steps, world, rmax)
    if e2e:
        e2e["ms"] = rmax(e2e["ms"])
    tokens_per_step = w.batch * N * world

    result = None
    if rank == 0:
        pk = peaks()
        counters = load_counters()
        alg = algorithmic_bytes(w, N, nnz_phi, nnz_psi, E)
        es = 2 if w.dtype == "bf16" else 4
        if mhat:   # Q, K, V read once, out written once; the mask blocks written once, read once
            mbytes = B.grf_mask_stats(feat.handle)[2]
            alg["mhat_attention"] = w.G * N * (2 * w.m + 2 * w.d) * es + mbytes
            alg["mask_build"] = mbytes + 2 * (nnz_phi + nnz_psi) * 8
        if asym:   # Q, K, V, Phi read once, out written once; no states
            alg["gather_contract"] = w.G * N * (2 * w.m + 2 * w.d) * es + nnz_phi * 8 + (N + 1) * 4
        per_kernel = {}
        for name, (ms, n) in ktimes.items():
            if n == 0:
                continue
            per = ms / n
            a = alg.get(name, 0)
            per_kernel[name] = {"ms_per_step": ms / steps, "launch_groups": n, "algorithmic_gb": a / 1e9,
                                "achieved_gbs": a / 1e9 / (per * 1e-3), "hbm_frac": a / 1e9 / (per * 1e-3) / pk["hbm_gbs"]}
        dom = max(ktimes, key=lambda kname: ktimes[kname][0])
        dom_ms = ktimes[dom][0] / max(ktimes[dom][1], 1)
        achieved = alg.get(dom, 0) / 1e9 / (dom_ms * 1e-3)
        binding = binding_report(w, N, nnz_phi, nnz_psi, ktimes, steps, pk, counters, plan_entries, mask_entries)
        # DRAM traffic of the dominant kernel from the tracked profile of the same sources, scaled to this run's heads
        traffic = None
        c = counters.get(dom)
        if c and not c["stale"] and c["workload"] == w.name.split("-heads")[0]:
            if dom in ("walk_merge", "mask_build"):            # independent of the head count
                traffic = c["dram_bytes"]
            elif dom == "mhat_attention":                      # the mask is read once whatever the head count: no scaling rule
                traffic = c["dram_bytes"] if w.G == c["heads"] else None
            else:
                traffic = c["dram_bytes"] * w.G / c["heads"]
        binds = binding.get(dom, {}).get("binds")
        bound = {"tensor_issue": "tensor", "hbm": "hbm", "integer_issue": "alu"}.get(binds, "hbm" if binds is None else "smem")
        step_text = {"sz": "grf_sample (both ensembles) + grf_masked_linear_attn",
                     "mhat": "grf_sample (both ensembles) + grf_features_materialise + grf_masked_attn_mhat",
                     "asym": "grf_sample (f_psi = delta_0) + grf_masked_attn_asym (Alg. 2, %s similarity)"
                             % ("softmax" if args.softmax else "linear")}[route]
        result = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": total_ms / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": ("bf16" if w.dtype == "bf16" else "f32"), "dtype_note": DTYPE_NOTE[route] if w.dtype == "bf16" else "fp32 throughout",
            "data": "synthetic",
            "config": {"workload": w.name, "route": route, "N": N, "edges": E, "batch": w.batch, "heads": w.heads, "m": w.m,
                       "d": w.d, "n_walks": w.n_walks, "p_halt": w.p_halt, "max_len": w.max_len,
                       "nnz_phi": nnz_phi, "nnz_psi": nnz_psi,
                       "node_order": "as given" if "unsorted" in w.name else
                                     ("Morton order of the points" if "pointcloud" in w.name else "generator's order"),
                       "features": "frozen: sampled once before the timed region" if frozen else
                                   ("walks sampled once and kept; new coefficients every step (grf_remodulate)" if remodulate
                                    else "resampled every step"),
                       "l2": "256 MiB flush write between steps, outside the per-step events",
                       "step": step_text.replace("grf_sample (both ensembles)", "grf_remodulate") + ", walks kept" if remodulate else
                               step_text + (", attention only (features frozen)" if frozen else ", features resampled every step")},
            "clocks": clocks,
            "gpu_launches": launches,
            "e2e": None if not e2e else
                   {"value": tokens_per_step / (e2e["ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                    "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": e2e["ms"],
                    "entry_point": "grf_step_host" + (" after grf_ctx_prefer_mask_route" if mhat else "")},
            "roofline": {"kernel": dom, "bound": bound, "frac_of": "hbm (the metric's roofline)", "achieved": achieved,
                         "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"], "peak_source": pk["source"],
                         "traffic": traffic, "algorithmic_bytes": alg.get(dom, 0),
                         "algorithmic_bytes_per_token_head": alg.get(dom, 0) / (w.G * N), "ms_per_launch": dom_ms,
                         "binding_resource": binds,
                         "fraction_of_binding_peak": binding.get(dom, {}).get("fraction_of_binding_peak")},
            "binding": binding,
            "phases": {"sample_ms": statistics.mean(sample_ms), "attn_ms": statistics.mean(attn_ms),
                       "sample_ms_min_med_max": [min(sample_ms), statistics.median(sample_ms), max(sample_ms)],
                       "attn_ms_min_med_max": [min(attn_ms), statistics.median(attn_ms), max(attn_ms)],
                       "walks_per_s": None if (frozen or remodulate) else 2 * N * w.n_walks / (statistics.mean(sample_ms) * 1e-3),
                       "attn_tokens_per_s": w.batch * N / (statistics.mean(attn_ms) * 1e-3),
                       "attn_hbm_frac": (2 * w.G * N * w.m * w.d * es + w.G * N * (2 * w.m + 2 * w.d) * es) / 1e9 /
                                        (statistics.mean(attn_ms) * 1e-3) / pk["hbm_gbs"] if route == "sz" else None,
                       "wall_s_timed_region": wall},
            "kernels": per_kernel,
        }
        if with_cpu_baseline and world == 1:
            result["cpu_baseline"] = cpu_baseline(w, g, f)
    feat.free()
    ctx.close()
    del ws, out, flush, qd, kd, vd
    torch.cuda.empty_cache()
    return result


_POOL_STATE = {}


def _cpu_pool_init(phi, psit):
    import oracle
    _POOL_STATE["Phi"] = oracle.CSR(*phi)
    _POOL_STATE["PsiT"] = oracle.CSR(*psit)
    oracle._load()


def _cpu_attn_head(qkv):
    import oracle
    q, k, v = qkv
    t0 = time.perf_counter()
    oracle.attn_sparse(q, k, v, _POOL_STATE["Phi"], _POOL_STATE["PsiT"], with_abs=False)
    return time.perf_counter() - t0


def cpu_baseline(w, g, f, max_heads=None):
    """The oracle as it stands, timed on this host: the whole sampler (one thread: it is a serial program) and the
    S/z-route attention of the batch's problems, one oracle process per problem on the cores this process may use
    (a spawn pool; the problems are independent, the oracle itself is not changed or tuned).  When there are fewer
    cores than problems, or `max_heads` bounds the sample, only that many problems run and the attention time is
    scaled to the whole batch."""
    import multiprocessing as mp

    import oracle
    from workloads import configs, tensors
    cores_avail = len(os.sched_getaffinity(0))
    t0 = time.perf_counter()
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    t_sample = time.perf_counter() - t0
    heads = max(1, min(w.G, cores_avail, max_heads or w.G))
    q, k, v = tensors.qkv(heads, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    qf, kf, vf = tensors.widen(q), tensors.widen(k), tensors.widen(v)
    pack = lambda M: (M.rowptr, M.col, M.val, None, M.shape)
    with mp.get_context("spawn").Pool(heads, initializer=_cpu_pool_init, initargs=(pack(Phi), pack(PsiT))) as pool:
        pool.map(_cpu_noop, range(heads))                     # workers started and the oracle loaded before the clock
        t0 = time.perf_counter()
        per_head = pool.map(_cpu_attn_head, [(qf[h:h + 1], kf[h:h + 1], vf[h:h + 1]) for h in range(heads)], chunksize=1)
        t_wall = time.perf_counter() - t0
    t_attn = t_wall * (w.G / heads)
    step = t_sample + t_attn
    return {"value": w.batch * g.N / step, "unit": UNIT, "cores": heads, "cores_available": cores_avail, "kind": "oracle",
            "sample": f"full sampler on one core ({t_sample:.2f} s) + {heads} of {w.G} problems of the attention, one "
                      f"oracle process each ({t_wall:.2f} s wall, {statistics.mean(per_head):.2f} s per problem)"
                      + ("" if heads == w.G else f", attention time scaled by {w.G}/{heads}"),
            "sampler_s": t_sample, "attn_s": t_attn, "attn_s_per_problem_one_core": statistics.mean(per_head),
            "single_core_value": w.batch * g.N / (t_sample + statistics.mean(per_head) * w.G)}


def _cpu_noop(_):
    return 0


def run_reference(args):
    """The CPU oracle timed as the reference arm: K steps, each the whole sampler plus a bounded sample of the
    batch's problems (at most four, one process each), sized so that the run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    import oracle
    w = make_workload(args.workload)
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    warm = min(args.warmup, 1)
    for _ in range(warm):
        cpu_baseline(w, g, f, max_heads=4)
    t0 = time.perf_counter()
    vals = []
    for _ in range(args.steps):
        vals.append(cpu_baseline(w, g, f, max_heads=4))
        if time.perf_counter() - t0 > 240 and len(vals) >= 3:     # keep the arm within a few minutes
            break
    value = statistics.mean(x["value"] for x in vals)
    ms = w.batch * g.N / value * 1e3
    base = dict(vals[-1]); base["value"] = value
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
            "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "route": "sz", "N": g.N, "batch": w.batch, "heads": w.heads, "m": w.m, "d": w.d},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def flops_figure(args):
    """Sec. 4 "Time complexity": operation counts against the number of nodes on 1-D grids, n = 4 walkers,
    p_halt = 0.5, m = d = 8, the masked count averaged over 10 seeds (features sampled on the GPU)."""
    from paper_2410_03462_b200 import api, binding as B
    from workloads import graphs
    ctx = api.Context(int(os.environ.get("LOCAL_RANK", "0")))
    L = 8
    f = B.grf_deconvolve(0.5 ** np.arange(L + 1)).astype(np.float32)
    rows = []
    for k in range(6, 15):
        N = 1 << k
        dg = api.DeviceGraph(graphs.path_graph(N, 0.5))
        masked = []
        for seed in range(10):
            feat = api.sample(ctx, dg, seed, 4, 0.5, L, f)
            mk, lin, sm = B.grf_attn_flops(feat.handle, 8, 8)
            masked.append(mk)
            feat.free()
        rows.append({"N": N, "masked_mean": float(np.mean(masked)), "masked_std": float(np.std(masked)),
                     "unmasked_linear": lin, "softmax": sm})
    ctx.close()
    return rows


def loglog_slope(xs, ys):
    lx, ly = np.log(np.asarray(xs, float)), np.log(np.asarray(ys, float))
    return float(np.polyfit(lx, ly, 1)[0])


def run_suite(args):
    """All workloads on both symmetric routes, the unsorted point cloud, frozen and re-modulated features, the sweep 2^10..2^20 (sz
    route) with the fitted slopes, and the operation counts; writes <dir>/bench_suite.jsonl and <dir>/bench_suite.md."""
    os.makedirs(args.suite_dir, exist_ok=True)
    lines, md = [], []

    def run(name, route, frozen=False, steps=10, remodulate=False):
        from paper_2410_03462_b200 import binding as B
        case = f"{name}/{route}" + ("/frozen" if frozen else "") + ("/remodulated" if remodulate else "")
        try:
            r = measure(args, name, route, False,
                        route == "sz" and not frozen and not remodulate and name in ("pc32768", "vit", "pc4096"),
                        frozen=frozen, steps=steps, warmup=3, remodulate=remodulate)
        except B.GrfError as e:          # e.g. the materialised mask of a graph without locality exceeds its limit
            lines.append({"suite_case": case, "error": str(e)})
            md.append(f"| {case} | not run: {e} |")
            return None
        r["suite_case"] = case
        lines.append(r)
        return r

    md.append("| case | N | G | ms/step | sampler ms | attention ms | M tokens/s | G walks/s | dominant kernel | its ms | HBM frac | binds (fraction of that peak) |")
    md.append("|---|---|---|---|---|---|---|---|---|---|---|---|")

    def row(r):
        if r is None:
            return
        c, ph, rf = r["config"], r["phases"], r["roofline"]
        fb = rf.get("fraction_of_binding_peak")
        md.append(f"| {r['suite_case']} | {c['N']} | {c['batch'] * c['heads']} | {r['ms_per_step']:.3f} | {ph['sample_ms']:.3f} | "
                  f"{ph['attn_ms']:.3f} | {r['value'] / 1e6:.2f} | "
                  f"{'-' if ph['walks_per_s'] is None else format(ph['walks_per_s'] / 1e9, '.2f')} | {rf['kernel']} | "
                  f"{rf['ms_per_launch']:.3f} | {rf['frac']:.3f} | {rf['binding_resource']} ({'-' if fb is None else format(fb, '.2f')}) |")

    for name in ("tiny", "vit", "pc4096", "pc32768", "pc32768-unsorted"):
        row(run(name, "sz"))
        if name != "tiny":
            row(run(name, "sz", frozen=True))
            row(run(name, "mhat"))
            row(run(name, "mhat", frozen=True))
            if name in ("vit", "pc32768"):
                row(run(name, "sz", remodulate=True))
                row(run(name, "mhat", remodulate=True))
    sweep = []
    for k in range(10, 21):
        r = run(f"sweep{k}", "sz", steps=10 if k < 18 else 4)
        row(r)
        if r is not None:
            sweep.append(r)
    big = [r for r in sweep if r["config"]["N"] >= 1 << 14]
    Ns = [r["config"]["N"] for r in big]
    slopes = {"sampler": loglog_slope(Ns, [r["phases"]["sample_ms"] for r in big]),
              "attention": loglog_slope(Ns, [r["phases"]["attn_ms"] for r in big])}
    md.append("")
    md.append(f"Sweep (8-regular graphs, sz route), log-log slope of time against N for N >= 2^14: sampler "
              f"{slopes['sampler']:.3f}, attention {slopes['attention']:.3f} (1.0 = linear time).")
    md.append("Attention time per token-head (ns): " + ", ".join(
        f"2^{int(math.log2(r['config']['N']))}: {r['phases']['attn_ms'] * 1e6 / (r['config']['N'] * r['config']['heads']):.1f}"
        for r in sweep) + " (the per-problem records outgrow L2, 126 MB, between 2^13 and 2^15).")
    fl = flops_figure(args)
    md.append("")
    md.append("Operation counts (Sec. 4 \"Time complexity\": 1-D grids, n = 4, p_halt = 0.5, m = d = 8, 10 seeds):")
    md.append("")
    md.append("| N | GRF-masked linear (mean) | std | unmasked linear | softmax | masked / unmasked linear |")
    md.append("|---|---|---|---|---|---|")
    for x in fl:
        md.append(f"| {x['N']} | {x['masked_mean']:.0f} | {x['masked_std']:.0f} | {x['unmasked_linear']} | {x['softmax']} | "
                  f"{x['masked_mean'] / x['unmasked_linear']:.2f} |")
    md.append("")
    md.append(f"log-log slope of the masked count against N: {loglog_slope([x['N'] for x in fl], [x['masked_mean'] for x in fl]):.3f}; "
              f"of the softmax count: {loglog_slope([x['N'] for x in fl], [x['softmax'] for x in fl]):.3f}.")
    with open(os.path.join(args.suite_dir, "bench_suite.jsonl"), "w") as fh:
        for r in lines:
            fh.write(json.dumps(r) + "\n")
        fh.write(json.dumps({"sweep_slopes": slopes, "flops_figure": fl}) + "\n")
    with open(os.path.join(args.suite_dir, "bench_suite.md"), "w") as fh:
        fh.write("\n".join(md) + "\n")
    return {"suite": "done", "cases": len(lines), "sweep_slopes": slopes, "dir": args.suite_dir}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="pc32768")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--route", choices=["sz", "asym", "mhat"], default="sz",
                    help="sz: Alg. 1 through per-node states (the default and the headline); mhat: Eqs. 1-2 over the "
                         "materialised mask Phi Psi^T; asym: Alg. 2 (asymmetric features, Psi = I); the last two are "
                         "variants outside the headline metric")
    ap.add_argument("--frozen", action="store_true", help="features sampled (and prepared) once, outside the timed steps")
    ap.add_argument("--remodulate", action="store_true",
                    help="walks sampled once and kept; every timed step re-modulates them with new coefficients")
    ap.add_argument("--softmax", action="store_true", help="with --route asym: A_ij = exp(q_i . k_j)")
    ap.add_argument("--heads", type=int, default=0, help="override the workload's head count (profiling of a smaller case)")
    ap.add_argument("--no-other-routes", action="store_true", help="skip the short runs of the other routes beside the headline")
    ap.add_argument("--suite", action="store_true")
    ap.add_argument("--suite-dir", default=os.path.join(ROOT, "gpurun_out"))
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        res = run_reference(args)
    else:
        import torch
        import torch.distributed as dist
        world = int(os.environ.get("WORLD_SIZE", "1"))
        local = int(os.environ.get("LOCAL_RANK", "0"))
        if world != args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
        torch.cuda.set_device(local)
        if world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        if args.suite:
            res = run_suite(args)
        else:
            res = measure(args, args.workload, args.route, not args.no_cpu_baseline, True, frozen=args.frozen,
                          remodulate=args.remodulate)
            # beside the headline (the route through the per-node states, features resampled every step): the same
            # workload on the route over the materialised mask, and both routes with frozen features, in short runs
            if res is not None and world == 1 and args.route == "sz" and not args.frozen and not args.remodulate and not args.no_other_routes:
                w = make_workload(args.workload)
                if w.dtype == "bf16" and w.d == 64 and w.m in (16, 32, 64):
                    from paper_2410_03462_b200 import binding as B
                    others = {}
                    for name, route, frozen in (("mhat_resampled", "mhat", False), ("mhat_frozen", "mhat", True),
                                                ("sz_frozen", "sz", True), ("mhat_remodulated", "mhat", "remod"),
                                                ("sz_remodulated", "sz", "remod")):
                        try:
                            r = measure(args, args.workload, route, False, False, frozen=(frozen is True),
                                        remodulate=(frozen == "remod"), steps=min(args.steps, 10), warmup=3)
                        except B.GrfError as e:
                            others[name] = {"error": str(e)}
                            continue
                        others[name] = {"value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"],
                                        "attn_ms": r["phases"]["attn_ms"], "step": r["config"]["step"],
                                        "kernels_ms": {k: v["ms_per_step"] for k, v in r["kernels"].items()}}
                    res["other_routes"] = others
        if world > 1:
            dist.destroy_process_group()
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
