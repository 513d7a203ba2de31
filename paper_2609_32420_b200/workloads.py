"""Seeded synthetic video-DiT attention workloads.

This module only makes INPUTS (bf16 Q/K/V bit patterns, recompute-row flags and
the parameter records that describe a workload).  It holds none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
sides can draw identical bits from it.

The inputs stand in for the activations of real video diffusion transformers
(the paper serves Wan / LTX style backbones on prompt streams that are not
available offline): they have the shapes, block counts, ragged tails and the
frame-structured logits of spatiotemporal self-attention, nothing more.

bf16 values travel as ``numpy.uint16`` bit patterns (numpy has no bf16 type).
Random numbers come from numpy's counter-based Philox generator keyed by
(seed, tensor, batch, head), so any single head can be produced on its own.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Dict, Iterable, Optional, Tuple

import numpy as np

MODE_TOPK = 0
MODE_CUMMASS = 1


# --------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (storage conversion only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# workload records
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class BuildParams:
    """Selection rule of the connectivity builder (mirrors carnator_build_params)."""
    mode: int = MODE_TOPK
    keep_ratio: float = 0.25
    mass: float = 0.9
    window_frames: int = -1          # -1: none; r >= 0: frames [f_lo-r, f_hi+r] of the query block are always kept
    text_dense: int = 0              # 1: blocks holding a text token are dense rows and dense columns
    count_includes_forced: int = 1   # 1: k counts the forced blocks; 0: k applies to the non-forced candidates


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: int
    B: int
    H: int
    D: int
    n_text: int
    T: int
    Hg: int
    Wg: int
    block: int
    build: BuildParams
    recompute_frac: float
    structured: bool = True          # rank-8 per-frame shared component (weight 0.5)
    n_buffer: int = 0                # rows allocated per head (>= N); 0 -> N
    history_mask: bool = True        # mask is built from the separate "history" Q/K pair
    seed: int = 0

    @property
    def N(self) -> int:
        return self.n_text + self.T * self.Hg * self.Wg

    @property
    def Nbuf(self) -> int:
        return max(self.n_buffer, self.N)

    @property
    def nqb(self) -> int:
        return -(-self.N // self.block)

    @property
    def nkb(self) -> int:
        return -(-self.N // self.block)

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _w(name, cfg, **kw) -> Workload:
    return Workload(name=name, cfg=cfg, seed=cfg, **kw)


WORKLOADS: Dict[str, Workload] = {
    # cfg 1 -- small enough for a full CPU comparison in seconds
    "tiny": _w("tiny", 1, B=1, H=2, D=64, n_text=0, T=4, Hg=16, Wg=16, block=64,
               build=BuildParams(keep_ratio=0.30), recompute_frac=3 / 16,
               structured=False, history_mask=False),
    # cfg 2 -- Wan-1.3B-shaped 480p; 32760 tokens in a 32768-row buffer
    "wan1p3b_480p": _w("wan1p3b_480p", 2, B=1, H=12, D=128, n_text=0, T=21, Hg=30, Wg=52, block=128,
                       build=BuildParams(keep_ratio=0.25, window_frames=1, count_includes_forced=1),
                       recompute_frac=0.15, n_buffer=32768),
    # cfg 3 -- CogVideoX-5B-shaped joint attention, 226 text tokens first
    "cogvideox5b": _w("cogvideox5b", 3, B=1, H=48, D=64, n_text=226, T=13, Hg=30, Wg=45, block=128,
                      build=BuildParams(keep_ratio=0.35, text_dense=1, count_includes_forced=0),
                      recompute_frac=0.20),
    # cfg 4 -- Wan-14B-shaped 720p (the configuration the headline metric is quoted on)
    "wan14b_720p": _w("wan14b_720p", 4, B=1, H=40, D=128, n_text=0, T=21, Hg=45, Wg=80, block=128,
                      build=BuildParams(keep_ratio=0.15, window_frames=1, count_includes_forced=1),
                      recompute_frac=0.10),
    # cfg 5 -- HunyuanVideo-shaped 720p / 129 frames, 256 text tokens first; density is swept
    "hunyuan_720p": _w("hunyuan_720p", 5, B=1, H=24, D=128, n_text=256, T=33, Hg=45, Wg=80, block=128,
                       build=BuildParams(keep_ratio=0.25, text_dense=1, count_includes_forced=0),
                       recompute_frac=0.10),
}

HUNYUAN_DENSITIES = (0.05, 0.10, 0.25, 0.50, 1.00)


def get(name: str) -> Workload:
    return WORKLOADS[name]


def shrunk(w: Workload, H: Optional[int] = None, T: Optional[int] = None,
           Hg: Optional[int] = None, Wg: Optional[int] = None) -> Workload:
    """Same recipe on a smaller grid / fewer heads (parity cases the CPU side finishes quickly)."""
    kw = {}
    if H is not None:
        kw["H"] = H
    if T is not None:
        kw["T"] = T
    if Hg is not None:
        kw["Hg"] = Hg
    if Wg is not None:
        kw["Wg"] = Wg
    w2 = w.replace(**kw)
    if w.n_buffer:
        # keep the "N valid rows in a longer zero-padded buffer" property
        w2 = w2.replace(n_buffer=(w2.N // 128 + 1) * 128)
    return w2.replace(name=w.name + "_shrunk")


# --------------------------------------------------------------------------
# generators
# --------------------------------------------------------------------------
_TENSOR_ID = {"Q": 0, "K": 1, "V": 2}


def _rng(seed: int, stream: int, b: int, h: int) -> np.random.Generator:
    key = np.array([np.uint64(seed) * np.uint64(1000003) + np.uint64(stream),
                    (np.uint64(b) << np.uint64(32)) | np.uint64(h)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _frame_component(w: Workload, tensor: str, b: int, h: int) -> Optional[np.ndarray]:
    """[T, D] fp32 shared per-frame offset: (0.5/sqrt(8)) * a_{h,f} @ W_h, rank 8.

    Q and K share the same component (same-frame logits get a positive bump and
    frame-to-frame affinity varies), V draws its own.  The component depends on
    the workload seed only, not on the target/history choice, so a historical
    request has the same structure and different noise.
    """
    if not w.structured:
        return None
    stream = 900 if tensor in ("Q", "K") else 901
    g = _rng(2000 * w.seed + 7, stream, b, h)
    Wh = g.standard_normal((8, w.D), dtype=np.float32)
    a = g.standard_normal((w.T, 8), dtype=np.float32)
    return (0.5 / math.sqrt(8.0)) * (a @ Wh)


def gen_head(w: Workload, tensor: str, b: int, h: int, which: str = "target") -> np.ndarray:
    """bf16 bits [Nbuf, D] of one head of Q, K or V.  Rows >= N are zero."""
    assert tensor in _TENSOR_ID and which in ("target", "history")
    noise_seed = 1000 * w.seed + (500 if which == "history" else 0)
    g = _rng(noise_seed, _TENSOR_ID[tensor], b, h)
    x = g.standard_normal((w.N, w.D), dtype=np.float32)
    c = _frame_component(w, tensor, b, h)
    if c is not None:
        hw = w.Hg * w.Wg
        vid = x[w.n_text:].reshape(w.T, hw, w.D)
        vid += c[:, None, :]
    out = np.zeros((w.Nbuf, w.D), dtype=np.uint16)
    out[: w.N] = f32_to_bf16_bits(x)
    return out


def gen_tensor(w: Workload, tensor: str, which: str = "target",
               heads: Optional[Iterable[Tuple[int, int]]] = None, threads: int = 1) -> np.ndarray:
    """bf16 bits [B, H, Nbuf, D].  With ``heads`` only those (b, h) are filled (others stay zero).
    Every head has its own generator, so ``threads`` > 1 fills heads concurrently with identical bits."""
    out = np.zeros((w.B, w.H, w.Nbuf, w.D), dtype=np.uint16)
    todo = list(heads) if heads is not None else [(b, h) for b in range(w.B) for h in range(w.H)]

    def one(bh):
        out[bh[0], bh[1]] = gen_head(w, tensor, bh[0], bh[1], which)
    if threads > 1 and len(todo) > 1:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, todo))
    else:
        for bh in todo:
            one(bh)
    return out


def gen_qkv(w: Workload, which: str = "target",
            heads: Optional[Iterable[Tuple[int, int]]] = None):
    hs = list(heads) if heads is not None else None
    return tuple(gen_tensor(w, t, which, hs) for t in ("Q", "K", "V"))


def text_blocks(w: Workload) -> int:
    """Number of leading blocks that hold at least one text token."""
    return -(-w.n_text // w.block) if w.n_text > 0 else 0


def gen_recompute_rows(w: Workload) -> np.ndarray:
    """uint8 [B, nqb]: seeded choice of round(frac * eligible) query blocks, video-only blocks eligible."""
    out = np.zeros((w.B, w.nqb), dtype=np.uint8)
    first = text_blocks(w)
    eligible = np.arange(first, w.nqb)
    n = int(round(w.recompute_frac * len(eligible)))
    for b in range(w.B):
        g = _rng(3000 * w.seed + 11, 950, b, 0)
        pick = g.choice(eligible, size=n, replace=False)
        out[b, pick] = 1
    return out


def gen_random_mask(w: Workload, density: float, seed: int = 0) -> np.ndarray:
    """uint8 [B, H, nqb, nkb] Bernoulli(density) mask (tests of the attention path on arbitrary masks)."""
    g = _rng(4000 * w.seed + seed, 960, 0, 0)
    return (g.random((w.B, w.H, w.nqb, w.nkb)) < density).astype(np.uint8)


def checksum(bits: np.ndarray) -> int:
    """Order-dependent 64-bit checksum of a bf16 bit buffer (recorded beside results)."""
    a = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint64).ravel()
    idx = (np.arange(a.size, dtype=np.uint64) % np.uint64(65521)) + np.uint64(1)
    return int((a * idx).sum(dtype=np.uint64))
