"""Pins for the region oracle (dilation radii 2 and 3 per frame, Chebyshev + smoothstep weights, latent
fusion, region-restricted connectivity)."""
import numpy as np

from oracle import carnator_oracle as orc
from tests.helpers import rand_bits


def _evidence(seed, T=3, H=9, W=11, p=0.04):
    rng = np.random.default_rng(seed)
    ev = rng.random((T, H, W)) < p
    ev[1] = False                      # a frame without evidence
    return ev


def test_single_token_gives_squares_and_known_weights():
    """One evidence token at (4,5) of a 9 x 11 frame: active = 5 x 5 square, context = 11 x 11 square clipped
    to the frame; weights: 1 at the token, 1 - s(1/2) = 1/2 on the first ring, 1 - s(1) = 0 on the second."""
    ev = np.zeros((1, 9, 11), dtype=bool)
    ev[0, 4, 5] = True
    active, context, W = orc.build_regions(ev, 2, 3)
    exp_active = np.zeros_like(ev); exp_active[0, 2:7, 3:8] = True
    assert np.array_equal(active, exp_active)
    assert context.all()                                   # radius 5 covers rows -1..9, columns 0..10
    assert W[0, 4, 5] == 1.0
    ring1 = np.zeros_like(ev); ring1[0, 3:6, 4:7] = True; ring1[0, 4, 5] = False
    np.testing.assert_allclose(W[ring1], 0.5)
    ring2 = exp_active & ~ring1 & ~ev
    np.testing.assert_allclose(W[ring2], 0.0)
    assert (W[~active] == 0).all()


def test_dilation_is_per_frame_nested_and_composes():
    ev = _evidence(1)
    active, context, W = orc.build_regions(ev, 2, 3)
    assert (ev <= active).all() and (active <= context).all()
    assert not active[1].any() and not context[1].any()    # nothing leaks across frames
    # square neighbourhoods compose: radius 2 then 3 == radius 5
    assert np.array_equal(context, orc.dilate_per_frame(ev, 5))
    # definition by brute force: within Chebyshev distance 2 of an evidence token of the same frame
    T, H, Wd = ev.shape
    for t in range(T):
        for y in range(H):
            for x in range(Wd):
                near = ev[t, max(0, y - 2):y + 3, max(0, x - 2):x + 3].any()
                assert active[t, y, x] == near
    assert ((W >= 0) & (W <= 1)).all() and (W[ev] == 1).all()


def test_band_normalisation_uses_largest_distance_in_band():
    """With radius 1 the band only holds distance 1, so d_hat = 1 and W = 0 on the whole band."""
    ev = _evidence(2)
    active, _, W = orc.build_regions(ev, 1, 3)
    band = active & ~ev
    assert band.any() and (W[band] == 0).all()


def test_fusion_endpoints_and_linearity():
    rng = np.random.default_rng(3)
    zt, zh = rng.standard_normal((4, 3, 9, 11)), rng.standard_normal((4, 3, 9, 11))
    _, _, W = orc.build_regions(_evidence(4), 2, 3)
    z = orc.fuse_latents(zt, zh, W)
    ev = W == 1.0
    out = W == 0.0
    np.testing.assert_array_equal(z[:, ev], zt[:, ev])
    np.testing.assert_array_equal(z[:, out], zh[:, out])
    half = W == 0.5
    np.testing.assert_allclose(z[:, half], 0.5 * (zt[:, half] + zh[:, half]))


def test_block_flags_text_first_token_order():
    region = np.zeros((2, 2, 4), dtype=bool)       # 16 video tokens
    region[1, 0, 3] = True                         # video token 8 + 3 = 11 -> token 5 + 11 = 16 with 5 text tokens
    f = orc.region_block_flags(region, n_text=5, block=4)
    assert f.tolist() == [1, 1, 0, 0, 1, 0]        # blocks 0,1 hold text; token 16 is in block 4
    assert orc.region_block_flags(region, 5, 4, text_value=0).tolist() == [0, 0, 0, 0, 1, 0]


def test_region_attention_is_intersection_and_skips_inactive_rows():
    rng = np.random.default_rng(5)
    N, D, b = 48, 8, 16
    Q, K, V = (rand_bits(rng, (1, 2, N, D)) for _ in range(3))
    mask = (rng.random((1, 2, 3, 3)) < 0.7).astype(np.uint8)
    mask[..., 0] = 1
    active_q = np.array([[1, 0, 1]], dtype=np.uint8)
    context_k = np.array([[1, 1, 0]], dtype=np.uint8)
    rows = [(0, h, I) for h in range(2) for I in range(3)]
    O, L = orc.attention_region_rows(Q, K, V, N, b, b, 0.3, mask, active_q, context_k, rows)
    eff = mask.copy(); eff[..., 2] = 0
    O2, L2 = orc.attention_rows(Q, K, V, N, b, b, 0.3, eff, None, rows)
    for r, (_, _, I) in enumerate(rows):
        if I == 1:
            assert np.isnan(O[r]).all() and np.isnan(L[r]).all()
        else:
            np.testing.assert_array_equal(O[r], O2[r])
            np.testing.assert_array_equal(L[r], L2[r])


def test_seed_expansion_matches_dense_softmax_matrix_and_invariants():
    """A taken from an explicitly materialised softmax matrix (every key), then the definition literally."""
    import math
    from tests.helpers import widen
    rng = np.random.default_rng(30)
    N, D, H = 40, 8, 3
    Q, K = rand_bits(rng, (1, H, N, D)), rand_bits(rng, (1, H, N, D))
    pos, neg = [3, 17, 22], [0, 5, 39, 11]
    S, per_head = orc.seed_expansion(Q, K, N, 0.4, pos, neg)
    q, k = widen(Q), widen(K)
    exp_heads = np.zeros((H, N))
    for h in range(H):
        for i in range(N):
            sc = [0.4 * float(q[0, h, i] @ k[0, h, j]) for j in range(N)]
            den = sum(math.exp(v) for v in sc)
            A = [math.exp(v) / den for v in sc]
            exp_heads[h, i] = max(A[u] for u in pos) - max(A[u] for u in neg)
    np.testing.assert_allclose(per_head[0], exp_heads, atol=1e-12)
    np.testing.assert_allclose(S[0], exp_heads.mean(axis=0), atol=1e-12)
    assert (np.abs(per_head) <= 1).all()
    S_same, _ = orc.seed_expansion(Q, K, N, 0.4, pos, pos)
    assert (S_same == 0).all()                                        # identical seed sets cancel
    S_all, _ = orc.seed_expansion(Q, K, N, 0.4, list(range(N)), neg)
    assert (S_all >= 0).all()                                         # max over every key dominates any subset
    S_empty, ph = orc.seed_expansion(Q, K, N, 0.4, pos, [])
    assert (ph > 0).all()
    # the sampled form (some heads, some query rows) gives the very entries of the full form and leaves the rest at 0
    rows = np.array([1, 7, 8, 39])
    _, ph_s = orc.seed_expansion(Q, K, N, 0.4, pos, neg, heads=[(0, 2), (0, 0)], rows=rows)
    np.testing.assert_allclose(ph_s[0, [0, 2]][:, rows], per_head[0, [0, 2]][:, rows], atol=1e-13)
    assert (ph_s[0, 1] == 0).all() and (np.delete(ph_s[0, 0], rows) == 0).all()
