"""GPU parity of carnator_build_connectivity against the builder oracle, through the C ABI.

Bar: the block mask is bit-exact except for blocks whose fp32 pooled score (the oracle's) lies
within 1e-4 of the row's selection threshold; always-kept blocks must match; in top-k mode the
per-row count must match.  Pooled scores themselves are compared to 2e-5 absolute.
"""
import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import to_dev
from tests.helpers import check_mask

pytestmark = pytest.mark.gpu


def _oracle(w, Qb, Kb, heads=None):
    bp = w.build
    return orc.build_connectivity(Qb, Kb, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, w.scale,
                                  bp.mode, bp.keep_ratio, bp.mass, bp.window_frames, bp.text_dense,
                                  bp.count_includes_forced, heads=heads)


def _gpu(w, Qb, Kb):
    Q, K = to_dev(Qb), to_dev(Kb)
    shape = cn.shape_of(w, Q, K)
    scores = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.float32, device="cuda")
    mask, ws = cn.build_connectivity(Q, K, shape, cn.params_of(w.build), pooled_scores=scores)
    assert cn.query_status(ws) == cn.OK
    return mask.cpu().numpy(), scores.cpu().numpy()


def _compare(w, Qb, Kb, heads=None, what=""):
    mask_g, scores_g = _gpu(w, Qb, Kb)
    mask_r, scores_r, theta, F = _oracle(w, Qb, Kb, heads)
    if heads is not None:
        sel = np.zeros((w.B, w.H), dtype=bool)
        for (b, h) in heads:
            sel[b, h] = True
        mask_g = np.where(sel[:, :, None, None], mask_g, 0)
        scores_g = np.where(sel[:, :, None, None], scores_g, 0)
    assert np.abs(scores_g - scores_r).max() <= 2e-5, f"{what}: pooled scores differ by {np.abs(scores_g - scores_r).max()}"
    return check_mask(mask_g, mask_r, scores_r, theta, F, topk_mode=(w.build.mode == wl.MODE_TOPK), what=what)


PATHS = [cn.BUILDER_THREE_KERNELS, cn.BUILDER_FUSED]
PATH_IDS = ["three_kernels", "fused"]


@pytest.fixture
def builder_path(request):
    """Small layers would take the three kernels by size; the parity cases below run on both paths."""
    cn.debug_set_builder_path(request.param)
    yield request.param
    cn.debug_set_builder_path(cn.BUILDER_AUTO)


@pytest.mark.parametrize("builder_path", PATHS, ids=PATH_IDS, indirect=True)
def test_tiny_topk(builder_path):
    w = wl.get("tiny")
    Qb, Kb, _ = wl.gen_qkv(w)
    _compare(w, Qb, Kb, what="tiny")


@pytest.mark.parametrize("builder_path", PATHS, ids=PATH_IDS, indirect=True)
@pytest.mark.parametrize("name,kw", [
    ("wan1p3b_480p", dict(H=2, T=3)),
    ("cogvideox5b", dict(H=3, T=2)),
    ("hunyuan_720p", dict(H=2, T=1)),
    ("hunyuan_720p", dict(H=2, T=28)),         # nkb = 790: four score tiles per row, 32 keys per lane
])
def test_midsize_window_text_rules(name, kw, builder_path):
    w = wl.shrunk(wl.get(name), **kw)
    Qb, Kb, _ = wl.gen_qkv(w, "history")
    _compare(w, Qb, Kb, what=name)


@pytest.mark.parametrize("mass", [0.5, 0.9, 0.95])
@pytest.mark.parametrize("name,kw", [("tiny", {}), ("wan1p3b_480p", dict(H=2, T=4))])
def test_cumulative_mass_mode(name, kw, mass):
    w = wl.get(name)
    if kw:
        w = wl.shrunk(w, **kw)
    w = w.replace(build=dataclasses.replace(w.build, mode=wl.MODE_CUMMASS, mass=mass))
    Qb, Kb, _ = wl.gen_qkv(w, "history")
    _compare(w, Qb, Kb, what=f"{name} cummass {mass}")


@pytest.mark.parametrize("builder_path", PATHS, ids=PATH_IDS, indirect=True)
def test_ties_are_broken_by_lower_block_index(builder_path):
    """Identical key blocks give identical pooled scores: the lower index must win, exactly as the oracle does."""
    w = wl.shrunk(wl.get("wan1p3b_480p"), H=1, T=2).replace(
        build=wl.BuildParams(keep_ratio=0.3, window_frames=-1))
    Qb, Kb, _ = wl.gen_qkv(w, "history")
    blk = Kb[:, :, :128].copy()
    for J in range(w.N // 128):
        Kb[:, :, J * 128:(J + 1) * 128] = blk
    mask_g, _ = _gpu(w, Qb, Kb)
    mask_r, _, _, _ = _oracle(w, Qb, Kb)
    full = w.N // 128
    np.testing.assert_array_equal(mask_g[..., :full], mask_r[..., :full])


@pytest.mark.parametrize("builder_path", PATHS, ids=PATH_IDS, indirect=True)
def test_keep_ratio_one_is_all_ones(builder_path):
    w = wl.shrunk(wl.get("hunyuan_720p"), H=1, T=1).replace()
    w = w.replace(build=dataclasses.replace(w.build, keep_ratio=1.0))
    Qb, Kb, _ = wl.gen_qkv(w, "history")
    mask_g, _ = _gpu(w, Qb, Kb)
    assert (mask_g == 1).all()


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("wan1p3b_480p", dict(H=3, T=5)), ("cogvideox5b", dict(H=5, T=3)),
                                     ("hunyuan_720p", dict(H=2, T=2)), ("wan14b_720p", dict(H=3)), ("hunyuan_720p", dict(H=2))])
def test_fused_kernel_and_three_kernel_path_agree(name, kw):
    """Large top-k layers run as one persistent kernel that pools and scores on the tensor cores (block means as three
    bf16 terms, six products per score, fp32 accumulate); the three separate kernels use CUDA-core fp32 sums and FFMA
    chains.  Both carry rounding errors of a few 1e-6 on scores of magnitude 3 to 4 (each is checked against the fp64
    oracle to 2e-5 elsewhere); masks may differ only where a score sits that close to the row's threshold."""
    w = wl.shrunk(wl.get(name), **kw) if kw else wl.get(name)
    nthreads = min(16, os.cpu_count() or 1)
    Q = to_dev(wl.gen_tensor(w, "Q", "history", threads=nthreads))
    K = to_dev(wl.gen_tensor(w, "K", "history", threads=nthreads))
    shape = cn.shape_of(w, Q, K)
    out = []
    try:
        for path in (cn.BUILDER_FUSED, cn.BUILDER_THREE_KERNELS):
            cn.debug_set_builder_path(path)
            scores = torch.full((w.B, w.H, w.nqb, w.nkb), float("nan"), dtype=torch.float32, device="cuda")
            mask, ws = cn.build_connectivity(Q, K, shape, cn.params_of(w.build), pooled_scores=scores)
            assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
            mask2, ws = cn.build_connectivity(Q, K, shape, cn.params_of(w.build), ws=ws)       # without the score output
            assert cn.query_status(ws) == cn.OK
            assert torch.equal(mask, mask2)
            out.append((mask, scores))
    finally:
        cn.debug_set_builder_path(cn.BUILDER_AUTO)
    (m0, s0), (m1, s1) = out
    assert float((s0 - s1).abs().max()) <= 1e-5
    assert bool((m0.sum(-1) == m1.sum(-1)).all())                       # top-k: same number of blocks per row
    assert int((m0 != m1).sum()) <= 1e-5 * m0.numel() + 2


# the HunyuanVideo-shaped layer also at the ends of its density sweep
FULL = [("wan1p3b_480p", None), ("cogvideox5b", None), ("wan14b_720p", None), ("hunyuan_720p", None),
        ("hunyuan_720p", 0.05), ("hunyuan_720p", 0.50)]


@pytest.mark.parametrize("name,keep", FULL, ids=[f[0] + ("" if f[1] is None else f"_{f[1]}") for f in FULL])
def test_full_size_masks_on_sampled_heads(name, keep):
    """Full-size launch; the oracle checks two heads in full (every row, every block)."""
    w = wl.get(name)
    if keep is not None:
        w = w.replace(build=dataclasses.replace(w.build, keep_ratio=keep))
    heads = [(0, 1), (0, w.H - 2)]
    nthreads = min(16, os.cpu_count() or 1)
    Qb = wl.gen_tensor(w, "Q", "history", threads=nthreads)
    Kb = wl.gen_tensor(w, "K", "history", threads=nthreads)
    n_excused = _compare(w, Qb, Kb, heads=heads, what=f"{name} keep={w.build.keep_ratio}")
    assert n_excused <= 8
