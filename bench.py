#!/usr/bin/env python
"""Benchmark of the block-sparse attention hot path on synthetic video-DiT-shaped inputs.

One step = one pass of the whole path over one batch: connectivity builder on the historical
Q/K pair (pool, score, select), mask compaction, sparse attention.  The headline value is the
effective TFLOP/s on computed tiles (4 * rows * cols * D per evaluated block pair) over the whole
step; ms per attention layer is reported beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--density R]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample of the same workload

Under torchrun (N > 1) every rank runs an independent replica of the workload on its own GPU
(the path has no exchange step); times are the max over ranks.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_32420_b200 import workloads as wl  # noqa: E402

METRIC = "effective TFLOP/s on computed tiles (ms per attention layer in ms_attn_layer)"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wan14b_720p", choices=list(wl.WORKLOADS))
    ap.add_argument("--density", type=float, default=None, help="override the builder's keep ratio")
    ap.add_argument("--attn-impl", default="auto", choices=["auto", "portable", "tcgen05"])
    ap.add_argument("--heads", type=int, default=None, help="run a slice with fewer heads (profiling captures)")
    ap.add_argument("--exact-builder", action="store_true",
                    help="also time carnator_build_connectivity_exact (block masses on the tensor cores) on the history pair")
    ap.add_argument("--regions", action="store_true",
                    help="also time the region builder, latent fusion and the region-restricted attention form")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(bf16=float(p["bf16_tflops"]), bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    hbm=float(p["hbm_gbs"]), source="measured")
    return dict(bf16=1590.0, bf16_sustained=1400.0, hbm=6650.0, source="fallback")


def workload_from_args(args) -> wl.Workload:
    w = wl.get(args.workload)
    if args.density is not None:
        w = w.replace(build=dataclasses.replace(w.build, keep_ratio=args.density))
    if args.heads is not None:
        w = w.replace(H=args.heads, name=f"{w.name}[H={args.heads}]")
    return w


def gen_parallel(w, tensor, which):
    """All heads of one tensor, generated on a few host threads."""
    return wl.gen_tensor(w, tensor, which, threads=min(16, os.cpu_count() or 1))


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "25",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample(w, target_seconds, mask_head0, rec):
    """Times the oracle, as it stands, on a bounded sample of (head 0, query block) rows of the workload.
    Returns (TFLOP/s, seconds, description, threads)."""
    from oracle import carnator_oracle as orc
    heads = [(0, 0)]
    Qb, Kb, Vb = wl.gen_qkv(w, heads=heads)
    mask = np.zeros((w.B, w.H, w.nqb, w.nkb), dtype=np.uint8)
    mask[0, 0] = mask_head0
    rng = np.random.default_rng(1234)
    order = rng.permutation(w.nqb)
    done_rows, flops, t_used = [], 0.0, 0.0
    rq = np.minimum(w.block, w.N - np.arange(w.nqb) * w.block).astype(np.float64)
    eff = (mask[0, 0] != 0) | (rec[0] != 0)[:, None]
    t0 = time.perf_counter()
    for c0 in range(0, w.nqb, 8):               # batches of 8 query blocks until the time target is reached
        batch = [int(I) for I in order[c0:c0 + 8]]
        orc.attention_rows(Qb, Kb, Vb, w.N, w.block, w.block, w.scale, mask, rec, [(0, 0, I) for I in batch])
        done_rows += batch
        for I in batch:
            flops += 4.0 * w.D * rq[I] * float((eff[I] * rq).sum())
        t_used = time.perf_counter() - t0
        if t_used >= target_seconds:
            break
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    desc = f"{len(done_rows)} of {w.nqb} query blocks of head 0 (seeded order), {flops / 1e9:.1f} GFLOP of computed tiles"
    return flops / t_used / 1e12, t_used, desc, threads


def history_mask_head0(w):
    from oracle import carnator_oracle as orc
    heads = [(0, 0)]
    Qh = wl.gen_tensor(w, "Q", "history" if w.history_mask else "target", heads)
    Kh = wl.gen_tensor(w, "K", "history" if w.history_mask else "target", heads)
    bp = w.build
    mask, _, _, _ = orc.build_connectivity(Qh, Kh, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, w.scale,
                                           bp.mode, bp.keep_ratio, bp.mass, bp.window_frames, bp.text_dense,
                                           bp.count_includes_forced, heads=heads)
    return mask[0, 0]


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload_from_args(args)
    rec = wl.gen_recompute_rows(w)
    mh0 = history_mask_head0(w)
    per_step = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(w, min(per_step, 2.0), mh0, rec)
    vals, secs, desc, threads = [], [], "", 1
    for _ in range(args.steps):
        v, s, desc, threads = oracle_sample(w, per_step, mh0, rec)
        vals.append(v); secs.append(s)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "density": w.build.keep_ratio, "note": "each step is a bounded sample of the layer"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# rank reduction (replicas only: the data path has no collective; only the timings are reduced)
# ------------------------------------------------------------------------------------------------
def max_over_ranks(values, device=None):
    """Element-wise MAX over ranks of a list of floats (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_tflops(flops_per_replica: float, world: int, ms_per_step: float) -> float:
    """Every rank runs one replica of the workload; the job's throughput is all replicas' work over the slowest rank's time."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2609_32420_b200 import build as cbuild
    from paper_2609_32420_b200 import carnator as cn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0 or world == 1:
        cbuild.build_library()
    if world > 1:
        dist.barrier()
    cn.lib()

    w = workload_from_args(args)
    impl = {"auto": cn.IMPL_AUTO, "portable": cn.IMPL_PORTABLE, "tcgen05": cn.IMPL_TCGEN05}[args.attn_impl]
    peaks = load_peaks()
    dev = torch.device("cuda", local)

    def to_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    which = "history" if w.history_mask else "target"
    host = {}
    for t in "QKV":
        host[t] = gen_parallel(w, t, "target")
    host["Qh"] = gen_parallel(w, "Q", which)
    host["Kh"] = gen_parallel(w, "K", which)
    Q, K, V, Qh, Kh = (to_dev(host[k]) for k in ("Q", "K", "V", "Qh", "Kh"))
    rec_np = wl.gen_recompute_rows(w)
    rec = torch.from_numpy(rec_np).to(dev)

    shape = cn.shape_of(w, Q, K, V, None, attn_impl=impl)
    bshape = cn.shape_of(w, Qh, Kh)
    params = cn.params_of(w.build)
    O = torch.empty((w.B, w.H, w.N, w.D), dtype=torch.bfloat16, device=dev)
    shape.o_stride = type(shape.o_stride)(*O.stride()[:3])
    LSE = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    mask = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=dev)
    bws = torch.empty(cn.build_workspace_bytes(bshape, params), dtype=torch.uint8, device=dev)
    aws = torch.empty(cn.attn_workspace_bytes(shape), dtype=torch.uint8, device=dev)

    def step(ev=None):
        if ev: ev[0].record()
        cn.build_connectivity(Qh, Kh, bshape, params, mask=mask, ws=bws)
        if ev: ev[1].record()
        cn.compact_mask(mask, rec, shape, ws=aws)
        if ev: ev[2].record()
        cn.sparse_attn_compacted(Q, K, V, shape, aws, O=O, LSE=LSE)
        if ev: ev[3].record()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    st = cn.query_status(aws)
    if st != cn.OK:
        raise SystemExit(f"device status {st}: {cn.last_cuda_error()}")
    tiles = cn.compacted_tiles(shape, aws)
    mask_np = mask.cpu().numpy()
    from_mask = (mask_np != 0) | (rec_np != 0)[:, None, :, None]
    rq = np.minimum(w.block, w.N - np.arange(w.nqb) * w.block).astype(np.float64)
    flops = 4.0 * w.D * float(np.einsum("bhij,i,j->", from_mask.astype(np.float64), rq, rq))
    density = float(from_mask.mean())

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    launches0 = cn.kernel_launches()
    sync_all()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        step(evs[i])
    t_end.record()
    sync_all()
    clocks = sampler.stop()
    launches = cn.kernel_launches() - launches0
    total_ms = t_start.elapsed_time(t_end)
    ms_build = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    ms_compact = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    ms_attn = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    ms_attn_min = float(np.min([e[2].elapsed_time(e[3]) for e in evs]))
    total_ms, ms_attn = max_over_ranks([total_ms, ms_attn], dev)
    ms_step = total_ms / args.steps
    value = whole_job_tflops(flops, world, ms_step)

    # ---- optional: the exact block-mass builder (second pass over Q K^T with the dense run's LSE) --------
    exact = None
    if args.exact_builder:
        ones = torch.ones((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=dev)
        Vz = torch.zeros_like(Kh)
        hsh = cn.shape_of(w, Qh, Kh, Vz, None, attn_impl=impl)
        _, Lh, _ = cn.sparse_attn(Qh, Kh, Vz, ones, None, hsh)
        del Vz, ones
        xparams = cn.params_of(dataclasses.replace(w.build, mode=wl.MODE_CUMMASS))
        xmask = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=dev)
        xws = torch.empty(cn.exact_workspace_bytes(bshape), dtype=torch.uint8, device=dev)
        for _ in range(3):
            cn.build_connectivity_exact(Qh, Kh, Lh, bshape, xparams, mask=xmask, ws=xws)
        torch.cuda.synchronize()
        n_x = max(3, min(args.steps, 10))
        xe = [torch.cuda.Event(enable_timing=True) for _ in range(n_x + 1)]
        xe[0].record()
        for i in range(n_x):
            cn.build_connectivity_exact(Qh, Kh, Lh, bshape, xparams, mask=xmask, ws=xws)
            xe[i + 1].record()
        torch.cuda.synchronize()
        x_ms = float(np.mean([xe[i].elapsed_time(xe[i + 1]) for i in range(n_x)]))
        x_flops = 2.0 * w.B * w.H * float(w.N) * float(w.N) * w.D
        exact = {"ms": x_ms, "tflops": x_flops / (x_ms * 1e-3) / 1e12, "frac": x_flops / (x_ms * 1e-3) / 1e12 / peaks["bf16"],
                 "flops_per_launch": x_flops, "mass": w.build.mass, "density": float(xmask.float().mean()),
                 "status": cn.query_status(xws), "steps": n_x, "bound": "tensor", "peak": peaks["bf16"]}
        del Lh, xmask, xws

    # ---- optional: reuse regions, latent fusion, region-restricted attention ---------------------------------
    regions = None
    if args.regions:
        rng = np.random.default_rng(77)
        ev = np.zeros((w.T, w.Hg, w.Wg), dtype=np.uint8)
        cy, cx = w.Hg // 2, w.Wg // 2
        for t in range(w.T):                                   # one drifting object tube, about 6 % of each frame
            cy = int(np.clip(cy + rng.integers(-1, 2), 6, w.Hg - 7)); cx = int(np.clip(cx + rng.integers(-2, 3), 10, w.Wg - 11))
            ev[t, cy - 5:cy + 6, cx - 9:cx + 10] = 1
        evd = torch.from_numpy(ev).to(dev)

        def timed(fn, n=20):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(); e0.record()
            for _ in range(n):
                fn()
            e1.record(); torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n

        ms_regions = timed(lambda: cn.build_regions(evd, shape, 2, 3))
        act, ctx, Wt = cn.build_regions(evd, shape, 2, 3)
        C_lat = 64                                             # latent channels per token (16 x 2 x 2 patch)
        zt = torch.randn((C_lat, w.T * w.Hg * w.Wg), dtype=torch.float32, device=dev)
        zh = torch.randn_like(zt); zo = torch.empty_like(zt)
        ms_fuse = timed(lambda: cn.fuse_latents(zt, zh, Wt.reshape(-1), z_out=zo))
        fuse_bytes = 3.0 * zt.numel() * 4 + Wt.numel() * 4
        aq = cn.region_block_flags(act, shape, w.block, 1).reshape(1, -1).contiguous()
        ck = cn.region_block_flags(ctx, shape, w.block, 1).reshape(1, -1).contiguous()
        rws = torch.empty(cn.attn_workspace_bytes(shape), dtype=torch.uint8, device=dev)
        ms_rattn = timed(lambda: cn.sparse_attn_region(Q, K, V, mask, aq, ck, shape, O, LSE, ws=rws), n=5)
        rtiles = cn.compacted_tiles(shape, rws)
        regions = {"ms_build_regions": ms_regions, "ms_fuse_latents": ms_fuse,
                   "fuse_gbs": fuse_bytes / (ms_fuse * 1e-3) / 1e9, "fuse_frac_of_hbm": fuse_bytes / (ms_fuse * 1e-3) / 1e9 / peaks["hbm"],
                   "active_query_blocks": int(aq.sum()), "context_key_blocks": int(ck.sum()),
                   "ms_region_attn": ms_rattn, "region_tiles": rtiles,
                   "region_attn_tflops": rtiles * 4.0 * w.block * w.block * w.D / (ms_rattn * 1e-3) / 1e12}
        del zt, zh, zo, rws

    # ---- end to end through the host-buffer calls --------------------------------------------------
    e2e = None
    if not args.no_e2e:
        pin = {k: torch.from_numpy((np.ascontiguousarray(host[k][:, :, : w.N]) if w.Nbuf != w.N else host[k]).view(np.int16)).pin_memory()
               for k in ("Q", "K", "V", "Qh", "Kh")}
        hshape = cn.shape_of(w, attn_impl=impl)
        hmask = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8).pin_memory()
        hrec = torch.from_numpy(rec_np).pin_memory()
        hO = torch.empty((w.B, w.H, w.N, w.D), dtype=torch.int16).pin_memory()
        hL = torch.empty((w.B, w.H, w.N), dtype=torch.float32).pin_memory()
        del Qh, Kh
        arena = torch.empty(max(cn.attn_host_arena_bytes(hshape), cn.build_host_arena_bytes(hshape, params)),
                            dtype=torch.uint8, device=dev)

        def e2e_step():
            cn.build_connectivity_host(pin["Qh"], pin["Kh"], hshape, params, hmask, arena)
            cn.sparse_attn_host(pin["Q"], pin["K"], pin["V"], hmask, hrec, hshape, hO, hL, arena)

        n_e2e = max(1, min(args.steps, 5))
        e2e_step()
        sync_all()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        e2e_ms = 1e3 * (t1 - t0) / n_e2e
        e2e_ms = max_over_ranks([e2e_ms], dev)[0]
        tb = w.B * w.H * w.N * w.D * 2
        mb = w.B * w.H * w.nqb * w.nkb
        e2e = {"value": whole_job_tflops(flops, world, e2e_ms), "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "steps": n_e2e, "h2d_bytes_per_step": 5 * tb + mb + w.B * w.nqb,
               "d2h_bytes_per_step": mb + tb + w.B * w.H * w.N * 4,
               "note": "carnator_build_connectivity_host + carnator_sparse_attn_host, pinned host buffers"}
        same = bool((hmask.numpy() == mask_np).all())
        e2e["mask_equals_device_run"] = same

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -----------------------------------------------------------
    attn_tflops = flops / (ms_attn * 1e-3) / 1e12
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "attn_traffic.txt")
    if os.path.exists(tpath):
        base = w.name.split("[")[0]
        for ln in open(tpath):
            parts = ln.split()
            if len(parts) == 3 and parts[0] == base and int(parts[2]) > 0:
                traffic = float(parts[1]) * tiles / float(parts[2])
    roofline = {"bound": "tensor", "kernel": "sparse attention", "achieved": attn_tflops, "peak": peaks["bf16"],
                "unit": "TFLOP/s", "frac": attn_tflops / peaks["bf16"], "traffic": traffic,
                "peak_source": peaks["source"] + " bf16_tflops (burst)", "frac_of_sustained": attn_tflops / peaks["bf16_sustained"],
                "frac_of_nominal_2250": attn_tflops / 2250.0, "flops_per_launch": flops}
    qk_bytes = 2.0 * w.B * w.H * w.N * w.D * 2
    builder = {"bound": "hbm", "ms": ms_build, "achieved": qk_bytes / (ms_build * 1e-3) / 1e9, "peak": peaks["hbm"],
               "unit": "GB/s", "frac": qk_bytes / (ms_build * 1e-3) / 1e9 / peaks["hbm"], "bytes_per_launch": qk_bytes}

    cpu = None
    if not args.no_cpu_baseline:
        v, secs, desc, threads = oracle_sample(w, args.cpu_seconds, mask_np[0, 0], rec_np)
        cpu = {"value": v, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": desc, "seconds": secs}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "D": w.D, "block": w.block,
                   "keep_ratio": w.build.keep_ratio, "effective_density": density, "computed_tiles": tiles,
                   "l2": "inputs larger than L2 (no flush needed)", "attn_impl": args.attn_impl,
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "ms_attn_layer": ms_attn, "ms_attn_layer_min": ms_attn_min, "ms_compact": ms_compact, "ms_build": ms_build,
        "attn_tflops": attn_tflops, "clocks": clocks, "gpu_launches": int(launches),
        "roofline": roofline, "builder_roofline": builder, "cpu_baseline": cpu, "e2e": e2e,
    }
    if exact is not None:
        line["exact_builder"] = exact
    if regions is not None:
        line["regions"] = regions
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
