#!/usr/bin/env python
"""Benchmark of the GRF-masked linear-attention path: one step = sample the graph random features
(walks, merge, CSR, regrouping) and evaluate the masked attention (state build, gather-contract) for one
batch of synthetic inputs.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload pc32768] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs the same-sized, independently seeded batch
on its own GPU (the problems are independent: no data-path collective); the value is the sum of all
ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
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
# DRAM bytes (read + write) of one launch at the default workload, from the ncu capture summarised in
# profiles/kernels_pointcloud32768_2heads.md (taken with 2 of the 8 heads; traffic grows in proportion to the
# heads, so the figures are scaled by 4).  Set an entry to None when its kernel changes after the capture.
NCU_TRAFFIC_BYTES = {
    "pointcloud-gmm16-N32768": {
        "gather_contract": 4 * (1.133120e9 + 12.062208e6),
        "build_states": 4 * (0.062991e9 + 226.052096e6),
        "row_denominators": 4 * (0.037775e9 + 0.042496e6),
        "walk_merge": 0.005105e9 + 6.034688e6,
    }
}


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
        return float(p["hbm_gbs"]), "measured"
    return FALLBACK_PEAKS["hbm_gbs"], "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples every 100 ms while the timed region runs (read-only queries)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={device_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
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


def rank_seed(base: int, rank: int) -> int:
    """Every rank draws its own batch: same shapes, different values."""
    return base + rank


def aggregate_over_ranks(local_ms: float, tokens_per_rank_step: int, steps: int, world: int, reduce_max):
    """Whole-job throughput: all ranks' tokens over the slowest rank's device time."""
    total_ms = reduce_max(local_ms)
    return total_ms, tokens_per_rank_step * world * steps / (total_ms * 1e-3)


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2410_03462_b200 import api, binding as B
    from workloads import configs, tensors

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = make_workload(args.workload)
    if args.heads > 0:
        w.heads = args.heads
        w.name += f"-heads{args.heads}"
    g = w.graph()
    N, E = g.N, g.E
    asym = args.route == "asym"
    mhat = args.route == "mhat"
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
    ws_bytes = B.grf_attn_workspace_bytes(w.G, N, w.m, w.d, dt)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    out = torch.empty_like(vd)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    feat = api.Features(ctx, None)

    def attention():
        if mhat:
            B.grf_features_materialise(ctx.handle, feat.handle)
            B.grf_masked_attn_mhat(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt, qd, kd, vd, out, None)
        elif asym:
            B.grf_masked_attn_asym(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt,
                                   B.GRF_KERNEL_SOFTMAX if args.softmax else B.GRF_KERNEL_LINEAR, qd, kd, vd, out, None)
        else:
            B.grf_masked_linear_attn(ctx.handle, feat.handle, w.G, N, w.m, w.d, dt, qd, kd, vd, out, None, ws, ws_bytes)

    def step(i):
        feat.handle = B.grf_sample(ctx.handle, N, dg.rowptr, dg.col, dg.w, configs.WALK_SEED + i, w.n_walks, w.p_halt,
                                   w.max_len, f, f_psi, feat.handle)
        attention()

    sampler = ClockSampler(local) if rank == 0 else None
    B.grf_ctx_enable_timing(ctx.handle, True)      # per-kernel events exist before the timed region starts
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    B.grf_ctx_kernel_times(ctx.handle)             # discard the warm-up record

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K steps, each bracketed by CUDA events on the stream the kernels run on;
    # L2 is flushed between steps, outside the events
    launches0 = ctx.launches
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    ev_mid = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    t_wall0 = time.perf_counter()
    t_epoch0 = time.time()
    for i in range(args.steps):
        flush.zero_()
        evs[i][0].record()
        feat.handle = B.grf_sample(ctx.handle, N, dg.rowptr, dg.col, dg.w, configs.WALK_SEED + 1000 + i, w.n_walks,
                                   w.p_halt, w.max_len, f, f_psi, feat.handle)
        ev_mid[i].record()
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

    # ---- end to end through the host-buffer entry point (pinned host memory; copies inside the timing)
    qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
    oh = torch.empty_like(v).pin_memory()
    rp_h = torch.from_numpy(g.rowptr).pin_memory(); c_h = torch.from_numpy(g.col).pin_memory()
    w_h = torch.from_numpy(g.w).pin_memory()
    e2e_steps = max(2, min(args.steps, 5))

    def host_step(i):
        B.grf_step_host(ctx.handle, N, rp_h, c_h, w_h, configs.WALK_SEED + 2000 + i, w.n_walks, w.p_halt, w.max_len,
                        f, None, w.G, w.m, w.d, dt, qh, kh, vh, oh)

    e2e_ms = float("nan")
    if not asym and not mhat:
        host_step(0)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            host_step(1 + i)
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
    h2d = (rp_h.numel() + c_h.numel() + w_h.numel()) * 4 + sum(t.numel() * t.element_size() for t in (qh, kh, vh))
    d2h = oh.numel() * oh.element_size()

    clocks = sampler.stop(t_epoch0, t_epoch1) if sampler else None

    # ---- max over ranks
    def rmax(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    total_ms, value = aggregate_over_ranks(total_ms, w.batch * N, args.steps, world, rmax)
    e2e_ms = rmax(e2e_ms)
    tokens_per_step = w.batch * N * world

    result = None
    if rank == 0:
        peak_gbs, peak_kind = peaks()
        alg = algorithmic_bytes(w, N, nnz_phi, nnz_psi, E)
        if mhat:   # Q, K, V read once, out written once, the mask blocks written once and read once
            es = 2
            mblocks, mentries, mbytes = B.grf_mask_stats(feat.handle)
            alg["mhat_attention"] = w.G * N * (2 * w.m + 2 * w.d) * es + mbytes
            alg["mask_build"] = mbytes + 2 * (nnz_phi + nnz_psi) * 8
        if asym:   # Q, K, V, Phi read once, out written once; no states
            es = 2 if w.dtype == "bf16" else 4
            alg["gather_contract"] = w.G * N * (2 * w.m + 2 * w.d) * es + nnz_phi * 8 + (N + 1) * 4
        per_kernel = {}
        for name, (ms, n) in ktimes.items():
            per = ms / max(n, 1)
            a = alg.get(name, 0)
            per_kernel[name] = {"ms_per_step": ms / args.steps, "launch_groups": n,
                                "algorithmic_gb": a / 1e9,
                                "achieved_gbs": a / 1e9 / (per * 1e-3) if n else None}
        dom = max(ktimes, key=lambda kname: ktimes[kname][0])
        dom_ms = ktimes[dom][0] / max(ktimes[dom][1], 1)
        achieved = alg.get(dom, 0) / 1e9 / (dom_ms * 1e-3)
        result = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 accumulate, " + w.dtype + " storage",
            "data": "synthetic",
            "config": {"workload": w.name, "N": N, "edges": E, "batch": w.batch, "heads": w.heads, "m": w.m, "d": w.d,
                       "n_walks": w.n_walks, "p_halt": w.p_halt, "max_len": w.max_len,
                       "nnz_phi": nnz_phi, "nnz_psi": nnz_psi,
                       "l2": "256 MiB flush write between steps, outside the per-step events",
                       "step": ("grf_sample (f_psi = delta_0) + grf_masked_attn_asym (Alg. 2, %s similarity), features "
                                "resampled every step" % ("softmax" if args.softmax else "linear")) if asym else
                               ("grf_sample (both ensembles) + grf_features_materialise + grf_masked_attn_mhat, features "
                                "resampled and the mask rebuilt every step") if mhat else
                               "grf_sample (both ensembles) + grf_masked_linear_attn, features resampled every step"},
            "clocks": clocks,
            "gpu_launches": launches,
            "e2e": None if (asym or mhat) else
                   {"value": tokens_per_step / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "entry_point": "grf_step_host"},
            "roofline": {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                         "frac": achieved / peak_gbs, "peak_source": peak_kind,
                         "traffic": None if (asym or mhat) else NCU_TRAFFIC_BYTES.get(w.name, {}).get(dom),
                         "algorithmic_bytes": alg.get(dom, 0), "ms_per_launch": dom_ms},
            "phases": {"sample_ms": statistics.mean(sample_ms), "attn_ms": statistics.mean(attn_ms),
                       "sample_ms_min_med_max": [min(sample_ms), statistics.median(sample_ms), max(sample_ms)],
                       "attn_ms_min_med_max": [min(attn_ms), statistics.median(attn_ms), max(attn_ms)],
                       "walks_per_s": 2 * N * w.n_walks / (statistics.mean(sample_ms) * 1e-3),
                       "attn_tokens_per_s": w.batch * N / (statistics.mean(attn_ms) * 1e-3),
                       "wall_s_timed_region": wall},
            "kernels": per_kernel,
        }
        if not args.no_cpu_baseline and world == 1:
            result["cpu_baseline"] = cpu_baseline(w, g, f, args.cpu_heads)
    feat.free()
    ctx.close()
    if world > 1:
        dist.destroy_process_group()
    return result


def cpu_baseline(w, g, f, heads: int = 1):
    """The oracle as it stands, timed on this host: the whole sampler plus `heads` of the batch's heads of
    the S/z-route attention; the step time is extrapolated linearly to all heads."""
    import oracle
    from workloads import configs, tensors
    t0 = time.perf_counter()
    Phi, Psi, PsiT, _, _ = oracle.sample(g.rowptr, g.col, g.w, configs.WALK_SEED, w.n_walks, w.p_halt, w.max_len, f)
    t_sample = time.perf_counter() - t0
    heads = max(1, min(heads, w.G))
    q, k, v = tensors.qkv(heads, g.N, w.m, w.d, w.dtype, configs.QKV_SEED)
    qf, kf, vf = tensors.widen(q), tensors.widen(k), tensors.widen(v)
    t0 = time.perf_counter()
    oracle.attn_sparse(qf, kf, vf, Phi, PsiT, with_abs=False)
    t_attn = (time.perf_counter() - t0) * (w.G / heads)
    step = t_sample + t_attn
    return {"value": w.batch * g.N / step, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"full sampler ({t_sample:.2f} s) + {heads} of {w.G} problems of the attention, "
                      f"attention time scaled by {w.G}/{heads} ({t_attn:.2f} s)",
            "sampler_s": t_sample, "attn_s_extrapolated": t_attn}


def run_reference(args):
    """The CPU oracle timed as the reference arm: K steps, each a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    import oracle
    w = make_workload(args.workload)
    g = w.graph()
    f = oracle.deconvolve(w.alpha).astype(np.float32)
    steps = max(1, min(args.steps, 3))
    for _ in range(min(args.warmup, 1)):
        cpu_baseline(w, g, f, 1)
    vals = [cpu_baseline(w, g, f, args.cpu_heads) for _ in range(steps)]
    value = statistics.mean(x["value"] for x in vals)
    ms = w.batch * g.N / value * 1e3
    base = dict(vals[-1]); base["value"] = value
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "N": g.N, "batch": w.batch, "heads": w.heads, "m": w.m, "d": w.d},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="pc32768")
    ap.add_argument("--cpu-heads", type=int, default=1, help="problems of the batch the CPU baseline really runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--route", choices=["sz", "asym", "mhat"], default="sz",
                    help="sz: Alg. 1 (per-node states, the default); asym: Alg. 2 (asymmetric features, Psi = I), "
                         "a variant outside the headline metric, no end-to-end leg")
    ap.add_argument("--softmax", action="store_true", help="with --route asym: A_ij = exp(q_i . k_j)")
    ap.add_argument("--heads", type=int, default=0, help="override the workload's head count (profiling of a smaller case)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    res = run_reference(args) if args.impl == "reference" else run_ours(args)
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
