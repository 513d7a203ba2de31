"""Pins for the attention oracle: none of these re-uses the oracle's own formula.

Each test is chosen so that a plausible mistake (dropped scale, wrong block ->
token mapping, tail keys not excluded, recompute flag ignored, transposed
operand, LSE in the wrong base) fails at least one of them.
"""
import math

import numpy as np
import pytest

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import workloads as wl
from tests.helpers import rand_bits, widen


def _case(seed, B=1, H=2, N=40, D=8, bq=16, bk=16, density=0.5, n_rec=1):
    rng = np.random.default_rng(seed)
    Q = rand_bits(rng, (B, H, N, D))
    K = rand_bits(rng, (B, H, N, D))
    V = rand_bits(rng, (B, H, N, D))
    nqb, nkb = -(-N // bq), -(-N // bk)
    mask = (rng.random((B, H, nqb, nkb)) < density).astype(np.uint8)
    rec = np.zeros((B, nqb), dtype=np.uint8)
    for b in range(B):
        rec[b, rng.choice(nqb, size=n_rec, replace=False)] = 1
    return Q, K, V, mask, rec


def test_hand_worked_case():
    """N=4, D=2, blocks of 2, scale 1.  Derivation (softmax by hand):
      q0=(1,0) sees keys 0,1: s=(0,1)      -> P=(1, e)/(1+e)
      q1=(0,1) sees keys 0,1: s=(0,0)      -> P=(1/2, 1/2)
      q2=(1,1) sees keys 0..3: s=(0,1,2,4) -> P=(1,e,e^2,e^4)/(1+e+e^2+e^4)
      q3=(0,0) sees keys 0..3: s=0         -> uniform over 4 keys
    """
    f = lambda a: wl.f32_to_bf16_bits(np.array(a, dtype=np.float32))[None, None]
    Q = f([[1, 0], [0, 1], [1, 1], [0, 0]])
    K = f([[0, 0], [1, 0], [0, 2], [2, 2]])
    V = f([[1, 0], [0, 1], [2, 2], [4, -4]])
    mask = np.array([[[[1, 0], [1, 1]]]], dtype=np.uint8)
    O, L = orc.attention_full(Q, K, V, 4, 2, 2, 1.0, mask)
    e = math.e
    den2 = 1 + e + e ** 2 + e ** 4
    exp_O = np.array([
        [1 / (1 + e), e / (1 + e)],
        [0.5, 0.5],
        [(1 + 2 * e ** 2 + 4 * e ** 4) / den2, (e + 2 * e ** 2 - 4 * e ** 4) / den2],
        [7 / 4, -1 / 4],
    ])
    exp_L = np.array([math.log(1 + e), math.log(2), math.log(den2), math.log(4)])
    np.testing.assert_allclose(O[0, 0], exp_O, rtol=0, atol=1e-12)
    np.testing.assert_allclose(L[0, 0], exp_L, rtol=0, atol=1e-12)


@pytest.mark.parametrize("seed,N,D,bq,bk", [(0, 40, 8, 16, 16), (1, 33, 4, 8, 16), (2, 48, 8, 16, 8)])
def test_matches_bruteforce_with_mask_tail_and_recompute(seed, N, D, bq, bk):
    Q, K, V, mask, rec = _case(seed, N=N, D=D, bq=bq, bk=bk)
    mask[0, 0, 1, :] = 0           # an empty row (unless it is the recompute row)
    scale = 1.0 / math.sqrt(D)
    O, L = orc.attention_full(Q, K, V, N, bq, bk, scale, mask, rec)
    Ob, Lb = orc.dense_bruteforce(Q, K, V, N, bq, bk, scale, mask, rec)
    np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
    assert np.array_equal(np.isneginf(L), np.isneginf(Lb))
    fin = np.isfinite(Lb)
    np.testing.assert_allclose(L[fin], Lb[fin], rtol=0, atol=1e-12)


def test_all_ones_mask_is_dense_softmax_attention():
    """Textbook dense attention written with a different library reduction (float64 softmax by hand)."""
    Q, K, V, mask, _ = _case(3, N=50, D=16, bq=16, bk=16)
    mask[:] = 1
    scale = 0.25
    O, L = orc.attention_full(Q, K, V, 50, 16, 16, scale, mask)
    q, k, v = widen(Q), widen(K), widen(V)
    s = np.einsum("bhid,bhjd->bhij", q, k) * scale
    w = np.exp(s - np.logaddexp.reduce(s, axis=-1, keepdims=True))
    np.testing.assert_allclose(O, np.einsum("bhij,bhjd->bhid", w, v), atol=1e-12)
    np.testing.assert_allclose(L, np.logaddexp.reduce(s, axis=-1), atol=1e-12)


def test_zero_queries_give_mean_of_allowed_values_and_log_count():
    """Q = 0 => P uniform on the allowed set => O = mean of allowed V rows, LSE = ln|allowed|.
    Pins the block -> token mapping, the ragged tail (N=43) and the recompute rows exactly."""
    N, bq, bk = 43, 16, 8
    Q, K, V, mask, rec = _case(4, N=N, D=8, bq=bq, bk=bk, density=0.4)
    Q[:] = 0
    mask[:, :, :, 0] = 1   # no empty rows here
    O, L = orc.attention_full(Q, K, V, N, bq, bk, 0.3, mask, rec)
    v = widen(V)
    for h in range(2):
        for i in range(N):
            I = i // bq
            cols = [j for j in range(N) if rec[0, I] or mask[0, h, I, j // bk]]
            np.testing.assert_allclose(O[0, h, i], v[0, h, cols].mean(axis=0), atol=1e-12)
            assert abs(L[0, h, i] - math.log(len(cols))) < 1e-12


def test_equal_keys_give_score_plus_log_count():
    """All key rows equal => every allowed score equals s_i => LSE_i = s_i + ln|allowed| (catches a wrong or missing scale)."""
    N, D, bq, bk = 37, 8, 16, 16
    Q, K, V, mask, rec = _case(5, N=N, D=D, bq=bq, bk=bk)
    mask[:, :, :, 1] = 1
    K[:] = K[:, :, :1]
    scale = 0.37
    _, L = orc.attention_full(Q, K, V, N, bq, bk, scale, mask, rec)
    q, k = widen(Q), widen(K)
    for h in range(2):
        for i in range(N):
            I = i // bq
            n_allowed = sum(1 for j in range(N) if rec[0, I] or mask[0, h, I, j // bk])
            s_i = scale * float(q[0, h, i] @ k[0, h, 0])
            assert abs(L[0, h, i] - (s_i + math.log(n_allowed))) < 1e-10


def test_rows_of_p_sum_to_one():
    """V = all ones => O = sum_j P_ij = 1 for every non-empty row."""
    Q, K, V, mask, rec = _case(6)
    mask[:, :, :, 2] = 1
    V[:] = wl.f32_to_bf16_bits(np.ones(1, dtype=np.float32))[0]
    O, _ = orc.attention_full(Q, K, V, 40, 16, 16, 0.35, mask, rec)
    np.testing.assert_allclose(O, 1.0, atol=1e-12)


def test_key_shift_invariance():
    """K_j += c for all j: O unchanged, LSE_i += scale * q_i . c (values chosen exact in bf16)."""
    N, D = 40, 8
    rng = np.random.default_rng(7)
    Q, K, V, mask, rec = _case(7, N=N, D=D)
    mask[:, :, :, 0] = 1
    kq = np.round(widen(K) * 8) / 8                 # multiples of 1/8, |x| small: exact in bf16
    c = np.round(rng.standard_normal(D) * 4) / 4
    K1 = wl.f32_to_bf16_bits(kq.astype(np.float32))
    K2 = wl.f32_to_bf16_bits((kq + c).astype(np.float32))
    assert np.array_equal(widen(K2), kq + c)
    scale = 0.5
    O1, L1 = orc.attention_full(Q, K1, V, N, 16, 16, scale, mask, rec)
    O2, L2 = orc.attention_full(Q, K2, V, N, 16, 16, scale, mask, rec)
    np.testing.assert_allclose(O1, O2, atol=1e-10)
    np.testing.assert_allclose(L2 - L1, scale * (widen(Q) @ c), atol=1e-10)


def test_merge_rule_for_disjoint_masks():
    """For disjoint key-block sets M1, M2: LSE = logaddexp(L1, L2) and O is the
    exp(LSE)-weighted mean -- the identity that gives LSE its meaning."""
    Q, K, V, mask, _ = _case(8, N=48, D=8, bq=16, bk=8, density=1.0)
    rng = np.random.default_rng(8)
    m1 = (rng.random(mask.shape) < 0.5).astype(np.uint8)
    m1[..., 0] = 1
    m2 = 1 - m1
    m2[..., 0] = 0
    m2[..., 1] = 1
    m1[..., 1] = 0
    args = (Q, K, V, 48, 16, 8, 0.4)
    O1, L1 = orc.attention_full(*args, m1)
    O2, L2 = orc.attention_full(*args, m2)
    O, L = orc.attention_full(*args, m1 | m2)
    np.testing.assert_allclose(L, np.logaddexp(L1, L2), atol=1e-12)
    w1, w2 = np.exp(L1 - L)[..., None], np.exp(L2 - L)[..., None]
    np.testing.assert_allclose(O, w1 * O1 + w2 * O2, atol=1e-12)
    # adding key blocks can only raise LSE
    assert (L >= L1 - 1e-12).all()


def test_single_block_equals_dense_attention_on_that_slice():
    Q, K, V, mask, _ = _case(9, N=48, D=8, bq=16, bk=16)
    mask[:] = 0
    mask[..., 2] = 1
    O, L = orc.attention_full(Q, K, V, 48, 16, 16, 0.3, mask)
    ones = np.ones((1, 2, 3, 1), dtype=np.uint8)
    Os, Ls = orc.attention_full(Q, K[:, :, 32:48], V[:, :, 32:48], 16, 16, 16, 0.3, ones[:, :, :1])
    np.testing.assert_allclose(O[:, :, :16], Os, atol=1e-12)
    np.testing.assert_allclose(L[:, :, :16], Ls, atol=1e-12)


def test_key_block_permutation_with_mask_columns():
    Q, K, V, mask, rec = _case(10, N=48, D=8, bq=16, bk=16)
    mask[..., 0] = 1
    perm = np.array([2, 0, 1])
    tok = np.concatenate([np.arange(16) + 16 * p for p in perm])
    O1, L1 = orc.attention_full(Q, K, V, 48, 16, 16, 0.3, mask, rec)
    O2, L2 = orc.attention_full(Q, K[:, :, tok], V[:, :, tok], 48, 16, 16, 0.3, mask[..., perm], rec)
    np.testing.assert_allclose(O1, O2, atol=1e-12)
    np.testing.assert_allclose(L1, L2, atol=1e-12)


def test_recompute_row_ignores_mask_contents():
    Q, K, V, mask, rec = _case(11, n_rec=2)
    O1, L1 = orc.attention_full(Q, K, V, 40, 16, 16, 0.3, mask, rec)
    ones = np.ones_like(mask)
    O2, L2 = orc.attention_full(Q, K, V, 40, 16, 16, 0.3, ones, None)
    for I in np.nonzero(rec[0])[0]:
        sl = slice(I * 16, min(40, (I + 1) * 16))
        np.testing.assert_allclose(O1[:, :, sl], O2[:, :, sl], atol=1e-13)
        np.testing.assert_allclose(L1[:, :, sl], L2[:, :, sl], atol=1e-13)


def test_empty_row_gives_zero_and_minus_inf():
    Q, K, V, mask, _ = _case(12)
    mask[0, 1, 2, :] = 0
    O, L = orc.attention_full(Q, K, V, 40, 16, 16, 0.3, mask, None)
    assert (O[0, 1, 32:40] == 0).all() and np.isneginf(L[0, 1, 32:40]).all()


def test_large_scores_stay_finite():
    Q, K, V, mask, rec = _case(13)
    mask[..., 0] = 1
    Q = wl.f32_to_bf16_bits((widen(Q) * 30).astype(np.float32))
    K = wl.f32_to_bf16_bits((widen(K) * 30).astype(np.float32))
    O, L = orc.attention_full(Q, K, V, 40, 16, 16, 1.0, mask, rec)
    assert np.isfinite(O).all() and np.isfinite(L).all()


def test_rows_api_matches_full_and_marks_tail_nan():
    Q, K, V, mask, rec = _case(14, N=40)
    O, L = orc.attention_full(Q, K, V, 40, 16, 16, 0.3, mask, rec)
    Or, Lr = orc.attention_rows(Q, K, V, 40, 16, 16, 0.3, mask, rec, [(0, 1, 2), (0, 0, 0)])
    np.testing.assert_array_equal(Or[0, :8], O[0, 1, 32:40])
    assert np.isnan(Or[0, 8:]).all() and np.isnan(Lr[0, 8:]).all()
    np.testing.assert_array_equal(Lr[1], L[0, 0, :16])


def test_tile_flop_count():
    mask = np.zeros((1, 1, 3, 3), dtype=np.uint8)
    mask[0, 0, 0, 0] = 1      # 16 x 16
    mask[0, 0, 2, 2] = 1      # 8 x 8 (tail)
    rec = np.array([[0, 1, 0]], dtype=np.uint8)   # row 1 dense: 16 x 40
    fl = orc.computed_tile_flops(40, 8, 16, 16, mask, rec)
    assert fl == 4 * 8 * (16 * 16 + 8 * 8 + 16 * 40)
