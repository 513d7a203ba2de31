"""Helpers for the GPU parity tests (device transfer, oracle row sampling)."""
import numpy as np
import torch

from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bits -> bf16 CUDA tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def o_to_host(O: torch.Tensor) -> np.ndarray:
    return O.float().cpu().numpy().astype(np.float64)


def tcgen05_available(shape) -> bool:
    return shape.block_q == 128 and shape.block_k == 128 and shape.D in (64, 128)


def impls_for(shape):
    out = [cn.IMPL_PORTABLE]
    if tcgen05_available(shape):
        out.append(cn.IMPL_TCGEN05)
    return out


def pick_rows(mask: np.ndarray, rec: np.ndarray, w, heads, extra_per_head=1, seed=0):
    """(b,h,I) rows for sampled comparison: per head a recompute row, the tail block, a text
    block (if any), the shortest and the longest masked row, plus random ones."""
    rng = np.random.default_rng(seed)
    rows = []
    for (b, h) in heads:
        cnt = mask[b, h].sum(-1).astype(np.int64)
        cnt_eff = np.where(rec[b] != 0, mask.shape[-1], cnt)
        pick = {int(w.nqb - 1), int(np.argmin(cnt_eff)), int(np.argmax(np.where(rec[b] != 0, -1, cnt)))}
        r = np.nonzero(rec[b])[0]
        if len(r):
            pick.add(int(r[0]))
        if w.n_text > 0:
            pick.add(0)
            pick.add(int(wl.text_blocks(w) - 1))
        for _ in range(extra_per_head):
            pick.add(int(rng.integers(0, w.nqb)))
        rows += [(b, h, I) for I in sorted(pick)]
    return rows


def gather_rows(O_gpu: torch.Tensor, L_gpu: torch.Tensor, rows, w):
    """GPU outputs for the listed (b,h,I) rows in the oracle's row layout (NaN past N)."""
    D = w.D
    O = np.full((len(rows), w.block, D), np.nan)
    L = np.full((len(rows), w.block), np.nan)
    for r, (b, h, I) in enumerate(rows):
        i0, i1 = I * w.block, min(w.N, (I + 1) * w.block)
        O[r, : i1 - i0] = O_gpu[b, h, i0:i1].float().cpu().numpy()
        L[r, : i1 - i0] = L_gpu[b, h, i0:i1].cpu().numpy()
    return O, L
