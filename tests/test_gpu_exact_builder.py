"""GPU parity of carnator_build_connectivity_exact (the paper's rule on exact block masses).

Checks, against the oracle and through the C ABI:
  1. block masses: |m_gpu - m_ref| <= 1e-3 * m_ref + 1e-6, rows sum to 1;
  2. selection: the GPU mask equals the oracle's selection rule applied to the GPU's own masses, exactly
     (same masses => same decisions, ties and always-kept blocks included);
  3. against the oracle's mask from its own fp64 masses: every row covers the target mass, and rows whose
     selection differs are rows where the oracle's kept mass crosses the target within 1e-3.
The LSE fed to the builder is the one a dense run of carnator_sparse_attn returns.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import to_dev
from tests.helpers import record

pytestmark = pytest.mark.gpu


def _dense_lse(w, Q, K):
    V = torch.zeros_like(Q)
    shape = cn.shape_of(w, Q, K, V)
    ones = torch.ones((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device="cuda")
    _, L, ws = cn.sparse_attn(Q, K, V, ones, None, shape)
    assert cn.query_status(ws) == cn.OK
    return L


def _run(w, mass, heads=None):
    Qb, Kb = wl.gen_tensor(w, "Q", "history"), wl.gen_tensor(w, "K", "history")
    Q, K = to_dev(Qb), to_dev(Kb)
    L = _dense_lse(w, Q, K)
    params = cn.params_of(dataclasses.replace(w.build, mode=wl.MODE_CUMMASS, mass=mass))
    bm = torch.empty((w.B, w.H, w.nqb, w.nkb), dtype=torch.float32, device="cuda")
    mask, ws = cn.build_connectivity_exact(Q, K, L, cn.shape_of(w, Q, K), params, block_mass=bm)
    assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
    return Qb, Kb, mask.cpu().numpy(), bm.cpu().numpy()


def _check(w, mass, Qb, Kb, mask_g, bm_g, heads, what):
    bp = w.build
    mask_r, bm_r, theta, F = orc.build_connectivity_exact(Qb, Kb, w.N, w.n_text, w.T, w.Hg, w.Wg, 128, 128, w.scale,
                                                          mass=mass, window_frames=bp.window_frames,
                                                          text_dense=bp.text_dense, heads=heads)
    n_rows = n_diff_rows = 0
    worst = 0.0
    for (b, h) in heads:
        mg, mr = bm_g[b, h].astype(np.float64), bm_r[b, h].astype(np.float64)
        err = np.abs(mg - mr)
        assert (err <= 1e-3 * mr + 1e-6).all(), f"{what}: block mass off by {err.max()}"
        worst = max(worst, float((err / (mr + 1e-6)).max()))
        np.testing.assert_allclose(mg.sum(-1), 1.0, atol=2e-3)
        for I in range(w.nqb):
            keep_self, _ = orc.select_by_mass(bm_g[b, h, I], F[I], mass)
            assert np.array_equal(mask_g[b, h, I] != 0, keep_self), f"{what}: selection differs from the rule on row {I}"
            n_rows += 1
            if not np.array_equal(mask_g[b, h, I], mask_r[b, h, I]):
                n_diff_rows += 1
                p = mr[I] / mr[I].sum()
                kept_r = p[mask_r[b, h, I] != 0].sum()
                last = p[np.nonzero((mask_r[b, h, I] != 0) & ~F[I])[0]].min() if ((mask_r[b, h, I] != 0) & ~F[I]).any() else 0.0
                t32 = float(np.float32(mass))
                assert min(abs(kept_r - t32), abs(kept_r - last - t32)) <= 1e-3, f"{what}: row {I} differs away from the threshold"
            assert (mg[I] / mg[I].sum())[mask_g[b, h, I] != 0].sum() >= float(np.float32(mass)) - 1e-6
    record("exact_mask", what, rows=n_rows, rows_differing=n_diff_rows, worst_rel_mass_err=worst,
           density=float(np.mean([mask_g[b, h].mean() for (b, h) in heads])))
    assert n_diff_rows <= max(2, n_rows // 100)


@pytest.mark.parametrize("name,kw,mass", [
    ("wan1p3b_480p", dict(H=2, T=3), 0.9),          # ragged tail, frame window
    ("cogvideox5b", dict(H=2, T=2), 0.8),           # D = 64, text rows / columns
    ("hunyuan_720p", dict(H=2, T=1), 0.95),
])
def test_exact_builder_midsize(name, kw, mass):
    w = wl.shrunk(wl.get(name), **kw)
    Qb, Kb, mask_g, bm_g = _run(w, mass)
    heads = [(0, h) for h in range(w.H)]
    _check(w, mass, Qb, Kb, mask_g, bm_g, heads, f"{name} exact mass={mass}")


def test_exact_builder_full_size_wan1p3b_sampled_head():
    w = wl.get("wan1p3b_480p")
    Qb, Kb, mask_g, bm_g = _run(w, 0.9)
    _check(w, 0.9, Qb, Kb, mask_g, bm_g, [(0, 5)], "wan1p3b_480p full exact mass=0.9")
