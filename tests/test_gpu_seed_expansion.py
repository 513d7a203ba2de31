"""GPU parity of carnator_seed_expansion against the oracle, through the C ABI.  The LSE is the one a dense run
of carnator_sparse_attn returns.  Values are attention probabilities in [0, 1]: pass if |d| <= 1e-3 * |ref| + 2e-6."""
import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw,n_pos,n_neg", [
    ("wan1p3b_480p", dict(H=3, T=3), 150, 333),      # ragged seed counts (not multiples of 64), ragged N
    ("cogvideox5b", dict(H=2, T=2), 64, 1),          # D = 64, text tokens present
    ("wan1p3b_480p", dict(H=1, T=2), 5, 0),          # empty background set
    ("wan1p3b_480p", dict(H=1, T=2), 0, 40),         # empty noun set
    ("wan1p3b_480p", dict(H=3, T=8), 192, 320),      # 512 seeds: both tensor-memory chunks full; CTAs whose tile range spans two heads
    ("wan1p3b_480p", dict(H=2, T=3), 300, 100),      # the set boundary falls inside a chunk and inside a group of 32 columns
    ("cogvideox5b", dict(H=5, T=6), 257, 255),       # D = 64, a boundary one past the first chunk
    ("wan1p3b_480p", dict(H=2, T=2), 400, 200),      # more seeds than the tensor-core form takes: the mma.sync kernel
])
def test_seed_expansion_matches_oracle(name, kw, n_pos, n_neg):
    w = wl.shrunk(wl.get(name), **kw)
    Qb, Kb = wl.gen_tensor(w, "Q"), wl.gen_tensor(w, "K")
    Q, K = to_dev(Qb), to_dev(Kb)
    V = torch.zeros_like(Q)
    shape = cn.shape_of(w, Q, K, V)
    ones = torch.ones((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device="cuda")
    _, L, ws = cn.sparse_attn(Q, K, V, ones, None, shape)
    assert cn.query_status(ws) == cn.OK
    rng = np.random.default_rng(n_pos + n_neg)
    tok = rng.choice(np.arange(w.n_text, w.N), size=n_pos + n_neg, replace=False).astype(np.int32)
    seeds = torch.from_numpy(tok).cuda()
    per_head = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device="cuda")
    out, sws = cn.seed_expansion(Q, K, L, seeds, n_pos, n_neg, cn.shape_of(w, Q, K), per_head=per_head, return_ws=True)
    if 0 < n_pos + n_neg <= 512:
        assert cn.query_status(sws) == cn.OK, cn.last_cuda_error()
    S_ref, ph_ref = orc.seed_expansion(Qb, Kb, w.N, w.scale, tok[:n_pos], tok[n_pos:])
    for got, ref in ((per_head.cpu().numpy(), ph_ref), (out.cpu().numpy(), S_ref)):
        assert (np.abs(got - ref) <= 1e-3 * np.abs(ref) + 2e-6).all(), float(np.abs(got - ref).max())


def test_full_size_layer_on_sampled_rows():
    """The Wan-14B-shaped layer in the launch configuration the bench times (one CTA per SM, about 160 query tiles
    each, most CTAs crossing a head boundary); the oracle checks 384 query rows of three heads, with its own
    softmax normaliser: every 128-row tile position, the ragged last tile and tiles next to head boundaries."""
    import os
    w = wl.get("wan14b_720p")
    nthreads = min(16, os.cpu_count() or 1)
    Qb, Kb = wl.gen_tensor(w, "Q", threads=nthreads), wl.gen_tensor(w, "K", threads=nthreads)
    Q, K = to_dev(Qb), to_dev(Kb)
    V = torch.zeros_like(Q)
    shape = cn.shape_of(w, Q, K, V)
    ones = torch.ones((w.B, w.H, w.nqb, w.nkb), dtype=torch.uint8, device="cuda")
    _, L, ws = cn.sparse_attn(Q, K, V, ones, None, shape)
    assert cn.query_status(ws) == cn.OK
    del V, ones
    n_pos, n_neg = 192, 320
    rng = np.random.default_rng(7)
    tok = rng.choice(np.arange(w.N), size=n_pos + n_neg, replace=False).astype(np.int32)
    per_head = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device="cuda")
    out, sws = cn.seed_expansion(Q, K, L, torch.from_numpy(tok).cuda(), n_pos, n_neg, cn.shape_of(w, Q, K),
                                 per_head=per_head, return_ws=True)
    assert cn.query_status(sws) == cn.OK, cn.last_cuda_error()
    heads = [(0, 0), (0, 17), (0, w.H - 1)]
    rows = np.unique(np.concatenate([rng.choice(w.N, size=320, replace=False), np.arange(0, 40),
                                     np.arange(w.N - 80, w.N), np.arange(128 * 300 - 8, 128 * 300 + 8)]))
    _, ph_ref = orc.seed_expansion(Qb, Kb, w.N, w.scale, tok[:n_pos], tok[n_pos:], heads=heads, rows=rows)
    got = per_head.cpu().numpy()
    for (b, h) in heads:
        g, r = got[b, h, rows], ph_ref[b, h, rows]
        assert (np.abs(g - r) <= 1e-3 * np.abs(r) + 2e-6).all(), (h, float(np.abs(g - r).max()))
    # the mean over heads is a plain reduction of per_head: check it against the GPU's own per-head values
    np.testing.assert_allclose(out.cpu().numpy(), got.mean(axis=1), rtol=1e-5, atol=1e-7)
