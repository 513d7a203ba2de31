#!/usr/bin/env python
"""Benchmark of the block-sparse attention hot path on synthetic video-DiT-shaped inputs.

One step = one pass of the whole path over one batch: connectivity builder on the historical
Q/K pair (pool, score, select), mask compaction, sparse attention.  The headline value is the
effective TFLOP/s on computed tiles (4 * rows * cols * D per evaluated block pair) over the whole
step; ms per attention layer is reported beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--density R] [--legs LIST]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample of the same workload

The same JSON line also carries the other measured claims (`--legs`, default all): `configs` (attention on the
other workload shapes), `density_sweep` (the HunyuanVideo-shaped layer at its five keep ratios with a least-squares
ns-per-tile fit), `exact_builder`, `regions`, `seed_expansion`; each leg samples the clocks for itself.

With N > 1 every rank runs an independent replica of the workload on its own GPU (the path has no exchange
step); times are the max over ranks.  `--gpus N` starts the N ranks by itself unless it already runs under
torchrun (WORLD_SIZE set).
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
    ap.add_argument("--legs", default=None,
                    help="comma list of extra legs: configs,density_sweep,exact_builder,regions,seed_expansion; 'none'; "
                         "default: all for the default workload with all heads, none otherwise")
    ap.add_argument("--exact-builder", action="store_true", help="same as adding exact_builder to --legs")
    ap.add_argument("--regions", action="store_true", help="same as adding regions to --legs")
    ap.add_argument("--selftest-launch", action="store_true", help=argparse.SUPPRESS)
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
    """Samples SM clock and throttle reasons with nvidia-smi while a timed region runs.

    One nvidia-smi process per GPU serves the whole run (its start-up takes longer than a short leg); every line is
    stamped with the host clock when it arrives, and a region takes the samples that fall between its start() and
    stop().  A region shorter than the sampling period takes the sample nearest to it and says so."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    PERIOD_MS = 25
    _shared = {}            # GPU index -> (process, list of (host time, line))

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.t0 = None

    @classmethod
    def _feed(cls, index):
        if index in cls._shared:
            return cls._shared[index]
        try:
            proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={cls.FIELDS}", "--format=csv,noheader,nounits", "-lms", str(cls.PERIOD_MS),
                 "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            cls._shared[index] = (None, [])
            return cls._shared[index]
        log = []

        def read():
            for line in proc.stdout:
                log.append((time.perf_counter(), line.strip()))
        threading.Thread(target=read, daemon=True).start()
        import atexit
        atexit.register(proc.terminate)
        cls._shared[index] = (proc, log)
        return cls._shared[index]

    def start(self):
        self.proc, self._log = self._feed(self.index)
        self.t0 = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        t1 = time.perf_counter()
        if self.t0 is not None:
            inside = [ln for (t, ln) in list(self._log) if self.t0 <= t <= t1 + 1e-3 * self.PERIOD_MS]
            how = "during"
            if not inside:              # region shorter than the sampling period: wait for the next sample
                deadline = time.perf_counter() + 0.5
                while time.perf_counter() < deadline and not any(t >= self.t0 for (t, _) in list(self._log)):
                    time.sleep(0.005)
                later = [ln for (t, ln) in list(self._log) if t >= self.t0]
                inside, how = later[:1], "first sample after the region"
            self.lines = inside
        else:
            how = "given"
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
                "power_w_max": max(power) if power else None, "samples": len(sm), "sampled": how,
                "reasons": sorted(reasons)}


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


def all_ranks(value, device=None):
    """Every rank's value, in rank order (a one-element list when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(value)]
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    out = [torch.zeros_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(out, t)
    return [float(o.item()) for o in out]


def whole_job_tflops(flops_per_replica: float, world: int, ms_per_step: float) -> float:
    """Every rank runs one replica of the workload; the job's throughput is all replicas' work over the slowest rank's time."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
ALL_LEGS = ("configs", "density_sweep", "exact_builder", "regions", "seed_expansion")
N_SM = 148
MUFU_PER_CLK_SM = 16          # exponentials per clock and SM (measured: 128 x 128 exponentials take 1024 clocks of one SM)


def legs_from_args(args):
    if args.legs is None:
        legs = set(ALL_LEGS) if (args.workload == "wan14b_720p" and args.heads is None and args.density is None) else set()
    elif args.legs.strip().lower() in ("none", ""):
        legs = set()
    elif args.legs.strip().lower() == "all":
        legs = set(ALL_LEGS)
    else:
        legs = {x.strip() for x in args.legs.split(",") if x.strip()}
        bad = legs - set(ALL_LEGS)
        if bad:
            raise SystemExit(f"unknown legs {sorted(bad)}; choose from {ALL_LEGS}")
    if args.exact_builder:
        legs.add("exact_builder")
    if args.regions:
        legs.add("regions")
    return legs


def mufu_bound_ms(tiles, block, sm_mhz):
    """Time the exponential unit alone needs for block x block exponentials per listed tile."""
    if not sm_mhz:
        return None
    return tiles * float(block) * block / (MUFU_PER_CLK_SM * N_SM * sm_mhz * 1e6) * 1e3


class Device:
    """Device-side state shared by the legs: binding, peaks, transfer helper, timing helper."""

    def __init__(self, local, impl, peaks):
        import torch
        from paper_2609_32420_b200 import carnator as cn
        self.torch, self.cn = torch, cn
        self.local, self.impl, self.peaks = local, impl, peaks
        self.dev = torch.device("cuda", local)

    def to_dev(self, bits):
        return self.torch.from_numpy(bits.view(np.int16)).to(self.dev).view(self.torch.bfloat16)

    def timed(self, fn, n, warm=3):
        """Mean ms of n calls after `warm` untimed ones, CUDA events on the current stream, clocks sampled meanwhile."""
        torch = self.torch
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        fn()
        torch.cuda.synchronize()
        once = max(time.perf_counter() - t0, 1e-6)
        n = int(min(2000, max(n, np.ceil(0.1 / once))))        # at least 0.1 s under load, so that the clocks are sampled
        sampler = ClockSampler(self.local)
        sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        ev[0].record()
        for i in range(n):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ts = [ev[i].elapsed_time(ev[i + 1]) for i in range(n)]
        return float(np.mean(ts)), float(np.min(ts)), clocks


def attention_leg(D, w, n, inputs=None, keep=None):
    """Builder on the history pair, compaction and attention of one workload; returns the timings of each and the
    roofline fractions of the attention kernel.  `inputs` carries device tensors between calls on the same workload."""
    torch, cn = D.torch, D.cn
    if keep is not None:
        w = w.replace(build=dataclasses.replace(w.build, keep_ratio=keep))
    if inputs is None:
        inputs = {}
    if "Q" not in inputs:
        which = "history" if w.history_mask else "target"
        for t in "QKV":
            inputs[t] = D.to_dev(gen_parallel(w, t, "target"))
        inputs["Qh"] = D.to_dev(gen_parallel(w, "Q", which))
        inputs["Kh"] = D.to_dev(gen_parallel(w, "K", which))
        inputs["rec_np"] = wl.gen_recompute_rows(w)
        inputs["rec"] = torch.from_numpy(inputs["rec_np"]).to(D.dev)
        inputs["O"] = torch.empty((w.B, w.H, w.N, w.D), dtype=torch.bfloat16, device=D.dev)
        inputs["LSE"] = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=D.dev)
        inputs["mask"] = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=D.dev)
    Q, K, V, Qh, Kh, O, LSE, mask, rec = (inputs[k] for k in ("Q", "K", "V", "Qh", "Kh", "O", "LSE", "mask", "rec"))
    shape = cn.shape_of(w, Q, K, V, None, attn_impl=D.impl)
    shape.o_stride = type(shape.o_stride)(*O.stride()[:3])
    bshape = cn.shape_of(w, Qh, Kh)
    params = cn.params_of(w.build)
    if "bws" not in inputs:
        inputs["bws"] = torch.empty(cn.build_workspace_bytes(bshape, params), dtype=torch.uint8, device=D.dev)
        inputs["aws"] = torch.empty(cn.attn_workspace_bytes(shape), dtype=torch.uint8, device=D.dev)
    bws, aws = inputs["bws"], inputs["aws"]
    ms_build, _, _ = D.timed(lambda: cn.build_connectivity(Qh, Kh, bshape, params, mask=mask, ws=bws), max(n, 5))
    ms_compact, _, _ = D.timed(lambda: cn.compact_mask(mask, rec, shape, ws=aws), max(n, 5))
    tiles = cn.compacted_tiles(shape, aws)
    ms_attn, ms_min, clocks = D.timed(lambda: cn.sparse_attn_compacted(Q, K, V, shape, aws, O=O, LSE=LSE), n)
    st = cn.query_status(aws)
    if st != cn.OK:
        raise SystemExit(f"{w.name}: device status {st}: {cn.last_cuda_error()}")
    from_mask = (mask.cpu().numpy() != 0) | (inputs["rec_np"] != 0)[:, None, :, None]
    rq = np.minimum(w.block, w.N - np.arange(w.nqb) * w.block).astype(np.float64)
    flops = 4.0 * w.D * float(np.einsum("bhij,i,j->", from_mask.astype(np.float64), rq, rq))
    tflops = flops / (ms_attn * 1e-3) / 1e12
    mufu = mufu_bound_ms(tiles, w.block, clocks.get("sm_mhz"))
    qk_bytes = 2.0 * w.B * w.H * w.N * w.D * 2
    out = {"workload": w.name, "H": w.H, "N": w.N, "D": w.D, "block": w.block, "keep_ratio": w.build.keep_ratio,
           "effective_density": float(from_mask.mean()), "computed_tiles": int(tiles), "flops": flops,
           "ms_attn": ms_attn, "ms_attn_min": ms_min, "ms_compact": ms_compact, "ms_build": ms_build,
           "attn_tflops": tflops, "frac_of_bf16_burst": tflops / D.peaks["bf16"],
           "frac_of_bf16_sustained": tflops / D.peaks["bf16_sustained"],
           "mufu_bound_ms": mufu, "frac_of_mufu_bound": (mufu / ms_attn) if mufu else None,
           "builder_gbs": qk_bytes / (ms_build * 1e-3) / 1e9, "builder_frac_of_hbm": qk_bytes / (ms_build * 1e-3) / 1e9 / D.peaks["hbm"],
           "executor": "tcgen05" if (w.block == 128 and D.impl != D.cn.IMPL_PORTABLE) else "portable (mma.sync)",
           "clocks": clocks}
    return out, inputs


def leg_configs(D, n):
    """Attention (and builder, compaction) on the other workload shapes; the HunyuanVideo-shaped one is in density_sweep."""
    out = []
    for name in ("tiny", "wan1p3b_480p", "cogvideox5b"):
        r, inputs = attention_leg(D, wl.get(name), n)
        out.append(r)
        del inputs
        D.torch.cuda.empty_cache()
    return out


def leg_density_sweep(D, n):
    """The HunyuanVideo-shaped layer at its five keep ratios: time against listed tiles, least-squares line."""
    w = wl.get("hunyuan_720p")
    inputs, pts = None, []
    for keep in wl.HUNYUAN_DENSITIES:
        r, inputs = attention_leg(D, w, n, inputs, keep=keep)
        pts.append(r)
    del inputs
    D.torch.cuda.empty_cache()
    x = np.array([p["computed_tiles"] for p in pts], dtype=np.float64)
    y = np.array([p["ms_attn"] for p in pts], dtype=np.float64)
    slope, intercept = np.polyfit(x, y, 1)
    resid = y - (slope * x + intercept)
    return {"workload": w.name, "points": pts, "ns_per_tile": slope * 1e6, "intercept_ms": float(intercept),
            "max_abs_residual_ms": float(np.abs(resid).max()),
            "ns_per_tile_at_each_point": [float(v) for v in (y / x * 1e6)]}


def leg_exact_builder(D, w, inputs, n):
    """carnator_build_connectivity_exact on the history pair (second pass over Q K^T with the dense run's LSE).  Every score
    costs one exponential and D multiply-adds on the tensor cores, so the exponential unit bounds the kernel."""
    torch, cn = D.torch, D.cn
    Qh, Kh = inputs["Qh"], inputs["Kh"]
    bshape = cn.shape_of(w, Qh, Kh)
    Lh = dense_lse(D, w, inputs)
    xparams = cn.params_of(dataclasses.replace(w.build, mode=wl.MODE_CUMMASS))
    xmask = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=D.dev)
    xws = torch.empty(cn.exact_workspace_bytes(bshape), dtype=torch.uint8, device=D.dev)
    ms, ms_min, clocks = D.timed(lambda: cn.build_connectivity_exact(Qh, Kh, Lh, bshape, xparams, mask=xmask, ws=xws), n)
    x_flops = 2.0 * w.B * w.H * float(w.N) * float(w.N) * w.D
    tiles = w.B * w.H * w.nqb * w.nkb
    # How the pooled-score estimator's mask (the one the timed steps run under) relates to the exact block masses of the
    # same history pair: reported, not a pass / fail (the paper prints no mask to compare with).
    bm = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.float32, device=D.dev)
    cn.build_connectivity_exact(Qh, Kh, Lh, bshape, xparams, mask=xmask, block_mass=bm, ws=xws)
    est = inputs["mask"] != 0
    exact = xmask != 0
    fidelity = {"estimator_mask_density": float(est.float().mean()),
                "attention_mass_under_estimator_mask": float((bm * est).sum(-1).mean()),
                "attention_mass_under_exact_mask": float((bm * exact).sum(-1).mean()),
                "estimator_recall_of_exact_mask": float((est & exact).sum() / exact.sum().clamp(min=1)),
                "exact_mask_recall_of_estimator": float((est & exact).sum() / est.sum().clamp(min=1))}
    del bm
    mufu = mufu_bound_ms(tiles, w.block, clocks.get("sm_mhz"))
    tf = x_flops / (ms * 1e-3) / 1e12
    return {"ms": ms, "ms_min": ms_min, "tflops": tf, "flops_per_launch": x_flops, "mass": w.build.mass,
            "density": float(xmask.float().mean()), "status": cn.query_status(xws),
            "bound": "exponential unit", "mufu_bound_ms": mufu, "frac_of_mufu_bound": (mufu / ms) if mufu else None,
            "frac_of_bf16_burst": tf / D.peaks["bf16"], "estimator_fidelity": fidelity, "clocks": clocks}


def dense_lse(D, w, inputs):
    """LSE of the history pair under an all-ones mask (shared by the exact builder and the seed expansion legs)."""
    torch, cn = D.torch, D.cn
    if "Lh" not in inputs:
        Qh, Kh = inputs["Qh"], inputs["Kh"]
        ones = torch.ones((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device=D.dev)
        Vz = torch.zeros_like(Kh)
        hsh = cn.shape_of(w, Qh, Kh, Vz, None, attn_impl=D.impl)
        _, inputs["Lh"], _ = cn.sparse_attn(Qh, Kh, Vz, ones, None, hsh)
        del Vz, ones
    return inputs["Lh"]


def leg_seed_expansion(D, w, inputs, n):
    """carnator_seed_expansion: Q is read once and multiplied by a few hundred gathered key rows per head."""
    torch, cn = D.torch, D.cn
    Qh, Kh = inputs["Qh"], inputs["Kh"]
    Lh = dense_lse(D, w, inputs)
    rng = np.random.default_rng(5)
    n_pos, n_neg = 192, 320
    tok = rng.choice(np.arange(w.n_text, w.N), size=n_pos + n_neg, replace=False).astype(np.int32)
    seeds = torch.from_numpy(tok).to(D.dev)
    shape = cn.shape_of(w, Qh, Kh)
    ws = torch.empty(cn.seed_workspace_bytes(shape), dtype=torch.uint8, device=D.dev)
    ms, ms_min, clocks = D.timed(lambda: cn.seed_expansion(Qh, Kh, Lh, seeds, n_pos, n_neg, shape, ws=ws), n)
    status = cn.query_status(ws)
    nbytes = float(w.B) * w.H * w.N * (w.D * 2 + 4 + 4) + float(w.B) * w.N * 4     # Q, LSE, per-head contrast, result
    flops = 2.0 * w.B * w.H * w.N * (n_pos + n_neg) * w.D                          # Q x K_seed^T
    return {"ms": ms, "ms_min": ms_min, "n_pos": n_pos, "n_neg": n_neg, "bytes_per_launch": nbytes, "flops_per_launch": flops,
            "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_hbm": nbytes / (ms * 1e-3) / 1e9 / D.peaks["hbm"],
            "tflops": flops / (ms * 1e-3) / 1e12, "frac_of_bf16_burst": flops / (ms * 1e-3) / 1e12 / D.peaks["bf16"],
            "bound": "tensor at this seed count; hbm (read Q once) below about 100 seeds",
            "executor": "tcgen05 (Q tile x 256 gathered seed key rows per product; gather kernel and head mean included)",
            "status": status, "clocks": clocks}


def leg_regions(D, w, inputs, n):
    """Region builder, latent fusion and the region-restricted attention form on the workload's grid."""
    torch, cn = D.torch, D.cn
    Q, K, V, O, LSE, mask = (inputs[k] for k in ("Q", "K", "V", "O", "LSE", "mask"))
    shape = cn.shape_of(w, Q, K, V, None, attn_impl=D.impl)
    shape.o_stride = type(shape.o_stride)(*O.stride()[:3])
    rng = np.random.default_rng(77)
    ev = np.zeros((w.T, w.Hg, w.Wg), dtype=np.uint8)
    cy, cx = w.Hg // 2, w.Wg // 2
    for t in range(w.T):                                   # one drifting object tube, about 6 % of each frame
        cy = int(np.clip(cy + rng.integers(-1, 2), 6, w.Hg - 7)); cx = int(np.clip(cx + rng.integers(-2, 3), 10, w.Wg - 11))
        ev[t, cy - 5:cy + 6, cx - 9:cx + 10] = 1
    evd = torch.from_numpy(ev).to(D.dev)
    ms_regions, _, _ = D.timed(lambda: cn.build_regions(evd, shape, 2, 3), 20)
    act, ctx, Wt = cn.build_regions(evd, shape, 2, 3)
    C_lat = 64                                             # latent channels per token (16 x 2 x 2 patch)
    zt = torch.randn((C_lat, w.T * w.Hg * w.Wg), dtype=torch.float32, device=D.dev)
    zh = torch.randn_like(zt); zo = torch.empty_like(zt)
    Wf = Wt.reshape(-1)
    ms_fuse, _, _ = D.timed(lambda: cn.fuse_latents(zt, zh, Wf, z_out=zo), 20)
    fuse_bytes = 3.0 * zt.numel() * 4 + Wt.numel() * 4
    aq = cn.region_block_flags(act, shape, w.block, 1).reshape(1, -1).contiguous()
    ck = cn.region_block_flags(ctx, shape, w.block, 1).reshape(1, -1).contiguous()
    rws = torch.empty(cn.attn_workspace_bytes(shape), dtype=torch.uint8, device=D.dev)
    ms_rattn, _, clocks = D.timed(lambda: cn.sparse_attn_region(Q, K, V, mask, aq, ck, shape, O, LSE, ws=rws), n)
    rtiles = cn.compacted_tiles(shape, rws)
    rt = rtiles * 4.0 * w.block * w.block * w.D / (ms_rattn * 1e-3) / 1e12
    return {"ms_build_regions": ms_regions, "ms_fuse_latents": ms_fuse, "fuse_bound": "hbm",
            "fuse_gbs": fuse_bytes / (ms_fuse * 1e-3) / 1e9, "fuse_frac_of_hbm": fuse_bytes / (ms_fuse * 1e-3) / 1e9 / D.peaks["hbm"],
            "active_query_blocks": int(aq.sum()), "context_key_blocks": int(ck.sum()),
            "ms_region_attn": ms_rattn, "region_tiles": rtiles, "region_attn_bound": "tensor",
            "region_attn_tflops": rt, "region_attn_frac_of_bf16_burst": rt / D.peaks["bf16"], "clocks": clocks}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2609_32420_b200 import build as cbuild
    from paper_2609_32420_b200 import carnator as cn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.selftest_launch:                     # CPU check of the launch path: gloo ranks, a stand-in step
        dist.init_process_group("gloo")
        ms = max_over_ranks([10.0 + 5.0 * rank])
        per_rank = all_ranks(10.0 + 5.0 * rank)
        if rank == 0:
            print(json.dumps({"selftest": True, "n_gpus": world, "ms_per_step": ms[0], "ms_per_rank": per_rank,
                              "config": {"parallelism": "replicas only"}}), flush=True)
        dist.destroy_process_group()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank}: no GPU {local} on this machine ({torch.cuda.device_count()} visible)")
    torch.cuda.set_device(local)
    ClockSampler._feed(local)                    # nvidia-smi takes a moment to start: long before the first timed region
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
    legs = legs_from_args(args)
    D = Device(local, impl, peaks)
    dev = D.dev
    to_dev = D.to_dev

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
    ms_per_rank = all_ranks(total_ms / args.steps, dev)
    total_ms, ms_attn = max_over_ranks([total_ms, ms_attn], dev)
    ms_step = total_ms / args.steps
    value = whole_job_tflops(flops, world, ms_step)

    # ---- extra legs that work on the headline workload's resident tensors (rank 0 reports them) -------------
    inputs = {"Q": Q, "K": K, "V": V, "Qh": Qh, "Kh": Kh, "O": O, "LSE": LSE, "mask": mask}
    n_leg = max(3, min(args.steps, 6))
    exact = leg_exact_builder(D, w, inputs, n_leg) if "exact_builder" in legs else None
    seed = leg_seed_expansion(D, w, inputs, n_leg) if "seed_expansion" in legs else None
    inputs.pop("Lh", None)
    regions = leg_regions(D, w, inputs, n_leg) if "regions" in legs else None

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
        inputs.pop("Qh"); inputs.pop("Kh")
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
        del arena, pin, hO, hL, hmask

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- legs on other workloads: release the headline tensors first ---------------------------------
    del Q, K, V, O, LSE, mask, inputs, bws, aws
    host.clear()
    torch.cuda.empty_cache()
    configs = leg_configs(D, n_leg) if "configs" in legs else None
    sweep = leg_density_sweep(D, n_leg) if "density_sweep" in legs else None

    # ---- roofline of the dominant kernel -----------------------------------------------------------
    attn_tflops = flops / (ms_attn * 1e-3) / 1e12
    traffic, traffic_src = None, None
    tpath = os.path.join(ROOT, "profiles", "attn_traffic.txt")
    if os.path.exists(tpath):
        base = w.name.split("[")[0]
        for ln in open(tpath):
            parts = ln.split()
            if len(parts) >= 3 and parts[0] == base and int(parts[2]) > 0:
                traffic = float(parts[1]) * tiles / float(parts[2])
                traffic_src = "profiles/attn_traffic.txt" + (f" (captured at {parts[3]})" if len(parts) > 3 else "")
    mufu = mufu_bound_ms(tiles, w.block, clocks.get("sm_mhz"))
    roofline = {"bound": "tensor", "kernel": "sparse attention", "achieved": attn_tflops, "peak": peaks["bf16"],
                "unit": "TFLOP/s", "frac": attn_tflops / peaks["bf16"], "traffic": traffic, "traffic_source": traffic_src,
                "peak_source": peaks["source"] + " bf16_tflops (burst)", "frac_of_sustained": attn_tflops / peaks["bf16_sustained"],
                "frac_of_nominal_2250": attn_tflops / 2250.0, "flops_per_launch": flops,
                "mufu_bound_ms": mufu, "frac_of_mufu_bound": (mufu / ms_attn) if mufu else None}
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
        "ms_per_rank": ms_per_rank,
        "ms_attn_layer": ms_attn, "ms_attn_layer_min": ms_attn_min, "ms_compact": ms_compact, "ms_build": ms_build,
        "attn_tflops": attn_tflops, "clocks": clocks, "gpu_launches": int(launches),
        "roofline": roofline, "builder_roofline": builder, "cpu_baseline": cpu, "e2e": e2e,
    }
    if configs is not None:
        line["configs"] = configs
    if sweep is not None:
        line["density_sweep"] = sweep
    if exact is not None:
        line["exact_builder"] = exact
    if regions is not None:
        line["regions"] = regions
    if seed is not None:
        line["seed_expansion"] = seed
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# --gpus N without torchrun: start the N replicas here
# ------------------------------------------------------------------------------------------------
def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_replicas(args) -> int:
    """Re-runs this command line as N ranks (one GPU each, rendezvous on 127.0.0.1) and passes rank 0's line through.
    The ranks are independent replicas; torch.distributed only carries the MAX of their timings."""
    n = args.gpus
    if not args.selftest_launch and args.impl == "ours":
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < n:
            sys.stderr.write(f"bench.py --gpus {n}: this machine shows {have} GPU(s); refusing to report fewer replicas than asked for\n")
            return 2
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    rc = procs[0].returncode
    for p in procs[1:]:
        p.wait()
        rc = rc or p.returncode
    sys.stdout.write(out)
    sys.stdout.flush()
    return rc


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.selftest_launch):
        raise SystemExit(launch_replicas(args))
    if args.impl == "reference" and not args.selftest_launch:
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
