"""GPU parity of the region kernels, latent fusion and the region-restricted attention form, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import o_to_host, to_dev
from tests.helpers import check_attention

pytestmark = pytest.mark.gpu


def _tube(T, H, W, seed, n_objects=2):
    """Evidence regions shaped like object tubes: a few drifting blobs, absent in some frames."""
    rng = np.random.default_rng(seed)
    ev = np.zeros((T, H, W), dtype=np.uint8)
    for o in range(n_objects):
        cy, cx = rng.integers(3, H - 3), rng.integers(3, W - 3)
        h, w = rng.integers(1, 5), rng.integers(1, 6)
        for t in range(T):
            if rng.random() < 0.15:
                continue
            cy = int(np.clip(cy + rng.integers(-1, 2), 0, H - 1)); cx = int(np.clip(cx + rng.integers(-1, 2), 0, W - 1))
            ev[t, max(0, cy - h):cy + h + 1, max(0, cx - w):cx + w + 1] = 1
    return ev


@pytest.mark.parametrize("T,H,W,ra,rc", [(5, 30, 52, 2, 3), (3, 17, 9, 2, 3), (2, 8, 8, 1, 4), (21, 45, 80, 2, 3)])
def test_regions_match_oracle(T, H, W, ra, rc):
    ev = _tube(T, H, W, seed=T * H + W)
    ev[T // 2] = 0
    shape = cn.make_shape(1, 1, T * H * W, 128, 0, T, H, W, 128, 128)
    a, c, Wt = cn.build_regions(torch.from_numpy(ev).cuda(), shape, ra, rc)
    a_ref, c_ref, W_ref = orc.build_regions(ev, ra, rc)
    np.testing.assert_array_equal(a.cpu().numpy() != 0, a_ref)          # integer work: bit-exact
    np.testing.assert_array_equal(c.cpu().numpy() != 0, c_ref)
    np.testing.assert_allclose(Wt.cpu().numpy(), W_ref, atol=1e-6)      # fp32 smoothstep of d / d_max, d in {1, 2}


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_latent_fusion_matches_oracle(dtype):
    T, H, W, C = 5, 30, 52, 16
    ev = _tube(T, H, W, seed=3)
    _, _, W_ref = orc.build_regions(ev, 2, 3)
    rng = np.random.default_rng(4)
    zt = torch.from_numpy(rng.standard_normal((C, T, H, W)).astype(np.float32)).to(dtype)
    zh = torch.from_numpy(rng.standard_normal((C, T, H, W)).astype(np.float32)).to(dtype)
    Wd = torch.from_numpy(W_ref.astype(np.float32)).cuda()
    out = cn.fuse_latents(zt.cuda(), zh.cuda(), Wd)
    ref = orc.fuse_latents(zt.float().numpy(), zh.float().numpy(), W_ref.astype(np.float32).astype(np.float64))
    got = out.float().cpu().numpy().astype(np.float64)
    if dtype == torch.float32:
        np.testing.assert_allclose(got, ref, atol=1e-6)
    else:                                                               # one bf16 rounding of the fp32 result
        assert (np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-6).all()
    # where W is exactly 1 or 0 the inputs pass through bit for bit
    assert torch.equal(out[:, Wd == 1], zt.cuda()[:, Wd == 1]) and torch.equal(out[:, Wd == 0], zh.cuda()[:, Wd == 0])


def test_block_flags_match_oracle():
    T, H, W, n_text = 3, 30, 45, 226
    ev = _tube(T, H, W, seed=9)
    shape = cn.make_shape(1, 1, n_text + T * H * W, 64, n_text, T, H, W, 128, 128)
    for tv in (0, 1):
        f = cn.region_block_flags(torch.from_numpy(ev).cuda(), shape, 128, tv)
        np.testing.assert_array_equal(f.cpu().numpy(), orc.region_block_flags(ev, n_text, 128, tv))


@pytest.mark.parametrize("impl,name,kw", [(cn.IMPL_TCGEN05, "wan1p3b_480p", dict(H=2, T=4)),
                                          (cn.IMPL_TCGEN05, "cogvideox5b", dict(H=2, T=2)),
                                          (cn.IMPL_PORTABLE, "wan1p3b_480p", dict(H=2, T=4))],
                         ids=["tcgen05_wan", "tcgen05_cog_text", "portable_wan"])
def test_region_restricted_attention_end_to_end(impl, name, kw):
    """evidence -> regions -> block flags -> attention restricted to active queries x context keys; inactive
    query blocks keep what the output buffer held (the cached values)."""
    w = wl.shrunk(wl.get(name), **kw)
    ev = _tube(w.T, w.Hg, w.Wg, seed=11, n_objects=1)
    dev_shape = cn.shape_of(w)
    a_dev, c_dev, _ = cn.build_regions(torch.from_numpy(ev).cuda(), dev_shape, 2, 3)
    active_q = cn.region_block_flags(a_dev, dev_shape, w.block, 1).reshape(1, -1).contiguous()
    context_k = cn.region_block_flags(c_dev, dev_shape, w.block, 1).reshape(1, -1).contiguous()
    a_ref, c_ref, _ = orc.build_regions(ev, 2, 3)
    aq = orc.region_block_flags(a_ref, w.n_text, w.block, 1)[None]
    ck = orc.region_block_flags(c_ref, w.n_text, w.block, 1)[None]
    np.testing.assert_array_equal(active_q.cpu().numpy(), aq)
    np.testing.assert_array_equal(context_k.cpu().numpy(), ck)
    assert 0 < aq.sum() < w.nqb                                  # some blocks active, some skipped

    Qb, Kb, Vb = wl.gen_qkv(w)
    mask = wl.gen_random_mask(w, 0.5, seed=2)
    mask[..., 0] = 1
    Q, K, V = to_dev(Qb), to_dev(Kb), to_dev(Vb)
    shape = cn.shape_of(w, Q, K, V, attn_impl=impl)
    O = torch.full((w.B, w.H, w.N, w.D), 3.0, dtype=torch.bfloat16, device="cuda")     # stands for the cached output
    L = torch.full((w.B, w.H, w.N), -7.0, dtype=torch.float32, device="cuda")
    ws = cn.sparse_attn_region(Q, K, V, torch.from_numpy(mask).cuda(), active_q, context_k, shape, O, L)
    assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
    rows = [(0, h, I) for h in range(w.H) for I in range(w.nqb)]
    O_ref, L_ref = orc.attention_region_rows(Qb, Kb, Vb, w.N, w.block, w.block, w.scale, mask, aq, ck, rows)
    O_ref = O_ref.reshape(1, w.H, w.nqb * w.block, w.D)[:, :, :w.N]
    L_ref = L_ref.reshape(1, w.H, w.nqb * w.block)[:, :, :w.N]
    skipped = np.isnan(L_ref)
    assert skipped.any() and (~skipped).any()
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, f"region {name}")
    Oh, Lh = O.float().cpu().numpy(), L.cpu().numpy()
    assert (Oh[skipped] == 3.0).all() and (Lh[skipped] == -7.0).all()
    eff = (mask != 0) & (aq != 0)[:, None, :, None] & (ck != 0)[:, None, None, :]
    assert cn.compacted_tiles(shape, ws) == int(eff.sum())
