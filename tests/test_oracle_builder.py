"""Pins for the connectivity-builder oracle (pooling, pooled scores, forced blocks, selection)."""
import math

import numpy as np
import pytest

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import workloads as wl
from tests.helpers import rand_bits, widen


def test_pooled_score_is_mean_of_score_tile():
    """Bilinearity: mean_i mean_j scale*q_i.k_j over a block pair == scale * q_bar . k_bar,
    with means over VALID tokens only (ragged tail N=45)."""
    rng = np.random.default_rng(0)
    N, D, bq, bk = 45, 8, 16, 8
    Q, K = rand_bits(rng, (N, D)), rand_bits(rng, (N, D))
    scale = 0.3
    S = orc.pooled_scores(Q, K, N, bq, bk, scale)
    q, k = widen(Q), widen(K)
    full = float(np.float32(scale)) * (q @ k.T)
    for I in range(-(-N // bq)):
        for J in range(-(-N // bk)):
            tile = full[I * bq: min(N, (I + 1) * bq), J * bk: min(N, (J + 1) * bk)]
            assert abs(float(S[I, J]) - tile.mean()) < 2e-6
    assert S.dtype == np.float32


def _forced_bruteforce(N, n_text, T, Hg, Wg, bq, bk, r, text_dense):
    """Per-token statement: a pair is forced if some query token and some key token of
    the two blocks satisfy the rule."""
    nqb, nkb = -(-N // bq), -(-N // bk)
    frame = [(-1 if t < n_text else (t - n_text) // (Hg * Wg)) for t in range(N)]
    F = np.zeros((nqb, nkb), dtype=bool)
    for I in range(nqb):
        qt = range(I * bq, min(N, (I + 1) * bq))
        for J in range(nkb):
            kt = range(J * bk, min(N, (J + 1) * bk))
            hit = False
            if text_dense and (any(frame[t] < 0 for t in qt) or any(frame[t] < 0 for t in kt)):
                hit = True
            if r >= 0 and not hit:
                qf = [frame[t] for t in qt if frame[t] >= 0]
                if qf:
                    lo, hi = min(qf) - r, max(qf) + r
                    hit = any(frame[t] >= 0 and lo <= frame[t] <= hi for t in kt)
            F[I, J] = hit
    return F


@pytest.mark.parametrize("n_text,T,Hg,Wg,bq,bk,r,td", [
    (0, 5, 3, 7, 16, 16, 1, 0),
    (0, 5, 3, 7, 16, 8, 0, 0),
    (10, 4, 5, 5, 16, 16, -1, 1),
    (10, 4, 5, 5, 8, 16, 1, 1),
    (20, 6, 2, 9, 16, 16, 2, 0),
])
def test_forced_blocks_match_per_token_rule(n_text, T, Hg, Wg, bq, bk, r, td):
    N = n_text + T * Hg * Wg
    F = orc.forced_blocks(N, n_text, T, Hg, Wg, bq, bk, r, td)
    np.testing.assert_array_equal(F, _forced_bruteforce(N, n_text, T, Hg, Wg, bq, bk, r, td))


def test_topk_count_values():
    assert orc.topk_count(0.30, 16) == 5          # ceil(4.8)
    assert orc.topk_count(0.25, 256) == 64        # exact product stays 64
    assert orc.topk_count(0.15, 591) == 89        # ceil(88.65)
    assert orc.topk_count(0.35, 137) == 48
    assert orc.topk_count(1.0, 931) == 931
    assert orc.topk_count(0.0001, 10) == 1        # never zero while a candidate exists
    assert orc.topk_count(0.5, 0) == 0


def test_topk_equals_stable_sort_and_order_invariants():
    rng = np.random.default_rng(1)
    for trial in range(50):
        n = int(rng.integers(1, 40))
        # coarse values => many ties
        s = (rng.integers(-3, 4, size=n) / 4).astype(np.float32)
        forced = rng.random(n) < 0.2
        for inc in (0, 1):
            ratio = float(rng.random())
            keep, theta = orc.select_topk(s, forced, ratio, inc)
            assert keep[forced].all()
            free = [j for j in range(n) if not forced[j]]
            if inc:
                n_admit = max(0, orc.topk_count(ratio, n) - int(forced.sum()))
            else:
                n_admit = orc.topk_count(ratio, len(free))
            n_admit = min(n_admit, len(free))
            ranked = sorted(free, key=lambda j: (-float(s[j]), j))     # python's sort: score desc, index asc
            expect = set(ranked[:n_admit]) | set(np.nonzero(forced)[0])
            assert set(np.nonzero(keep)[0]) == expect
            kept_free = [j for j in free if keep[j]]
            drop_free = [j for j in free if not keep[j]]
            if kept_free and drop_free:
                assert min(s[kept_free]) >= max(s[drop_free])
            if n_admit:
                assert theta == s[ranked[n_admit - 1]]
            else:
                assert np.isnan(theta)


def test_topk_against_library_topk_without_ties():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(2)
    s = rng.standard_normal(64).astype(np.float32)
    keep, theta = orc.select_topk(s, np.zeros(64, dtype=bool), 0.25, 1)
    vals, idx = torch.topk(torch.from_numpy(s), 16)
    assert set(np.nonzero(keep)[0]) == set(idx.tolist())
    assert theta == vals[-1].item()


def test_ratio_one_keeps_everything():
    s = np.random.default_rng(3).standard_normal(31).astype(np.float32)
    keep, _ = orc.select_topk(s, np.zeros(31, dtype=bool), 1.0, 0)
    assert keep.all()


def test_cummass_covers_mass_and_is_minimal():
    rng = np.random.default_rng(4)
    for trial in range(50):
        n = int(rng.integers(2, 40))
        s = (2.0 * rng.standard_normal(n)).astype(np.float32)
        forced = rng.random(n) < 0.15
        tau = float(rng.choice([0.5, 0.9, 0.95]))
        keep, theta = orc.select_cummass(s, forced, tau)
        p = np.exp(s.astype(np.float64) - s.max())
        p /= p.sum()
        tau32 = float(np.float32(tau))
        assert keep[forced].all()
        assert p[keep].sum() >= tau32 - 1e-12
        admitted = keep & ~forced
        if admitted.any():
            # minimal: dropping the weakest admitted block falls below the target
            weakest = min(np.nonzero(admitted)[0], key=lambda j: (float(s[j]), -j))
            assert p[keep].sum() - p[weakest] < tau32
            assert theta == s[weakest]
            # a descending prefix: nothing dropped outscores an admitted block
            dropped = ~keep
            if dropped.any():
                assert s[admitted].min() >= s[dropped].max()
        else:
            assert p[forced].sum() >= tau32 and np.isnan(theta)


def test_build_connectivity_tiny_workload_counts_and_planted_structure():
    w = wl.get("tiny")
    Q, K, _ = wl.gen_qkv(w)
    bp = w.build
    mask, scores, theta, F = orc.build_connectivity(
        Q, K, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, w.scale,
        bp.mode, bp.keep_ratio, bp.mass, bp.window_frames, bp.text_dense, bp.count_includes_forced)
    assert mask.shape == (1, 2, 16, 16) and (mask.sum(-1) == 5).all()
    assert not F.any()
    # the threshold is the smallest kept score of each row
    kept_min = np.where(mask != 0, scores, np.inf).min(-1)
    np.testing.assert_array_equal(kept_min, theta)


def test_build_connectivity_window_and_text_rules_on_structured_input():
    w = wl.shrunk(wl.get("cogvideox5b"), H=2, T=3, Hg=10, Wg=12).replace(
        n_text=40, block=32,
        build=wl.BuildParams(keep_ratio=0.35, window_frames=0, text_dense=1, count_includes_forced=0))
    Q, K, _ = wl.gen_qkv(w, "history")
    bp = w.build
    mask, scores, theta, F = orc.build_connectivity(
        Q, K, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, w.scale,
        bp.mode, bp.keep_ratio, bp.mass, bp.window_frames, bp.text_dense, bp.count_includes_forced)
    assert (mask[:, :, F] == 1).all()
    assert (mask[:, :, :2] == 1).all() and (mask[:, :, :, :2] == 1).all()   # 40 text tokens touch blocks 0, 1
    for I in range(2, w.nqb):
        n_free = int((~F[I]).sum())
        assert (mask[0, :, I].sum(-1) == F[I].sum() + orc.topk_count(0.35, n_free)).all()


def test_structured_inputs_make_same_frame_blocks_win():
    """Sanity of the input recipe, not parity: with the shared per-frame component the
    pooled score of same-frame block pairs is well above that of other pairs."""
    w = wl.shrunk(wl.get("wan1p3b_480p"), H=2, T=6, Hg=16, Wg=16)
    Q, K, _ = wl.gen_qkv(w, "history")
    S = orc.pooled_scores(Q[0, 0], K[0, 0], w.N, 128, 128, w.scale)
    same = np.kron(np.eye(6, dtype=bool), np.ones((2, 2), dtype=bool))     # 256 tokens/frame = 2 blocks
    assert S[same].mean() > S[~same].mean() + 1.0


def test_block_mass_rows_sum_to_one_and_estimator_recall_reported():
    w = wl.get("tiny")
    Q, K, _ = wl.gen_qkv(w)
    M = orc.block_mass_exact(Q[0, 0], K[0, 0], w.N, 64, 64, w.scale)
    np.testing.assert_allclose(M.sum(-1), 1.0, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# exact block-mass rule (the paper's literal statement)
# ---------------------------------------------------------------------------------------------
def _mass_bruteforce(Q, K, N, bq, bk, scale):
    q, k = widen(Q), widen(K)
    nqb, nkb = -(-N // bq), -(-N // bk)
    out = np.zeros((nqb, nkb))
    for i in range(N):
        s = [scale * sum(q[i, d] * k[j, d] for d in range(q.shape[1])) for j in range(N)]
        mx = max(s)
        den = sum(math.exp(v - mx) for v in s)
        for j in range(N):
            out[i // bq, j // bk] += math.exp(s[j] - mx) / den
    for I in range(nqb):
        out[I] /= min(bq, N - I * bq)
    return out


def test_block_mass_matches_bruteforce_and_rows_sum_to_one():
    rng = np.random.default_rng(20)
    N, D, bq, bk = 37, 4, 8, 16
    Q, K = rand_bits(rng, (N, D)), rand_bits(rng, (N, D))
    M = orc.block_mass_exact(Q, K, N, bq, bk, 0.7)
    np.testing.assert_allclose(M, _mass_bruteforce(Q, K, N, bq, bk, 0.7), atol=1e-12)
    np.testing.assert_allclose(M.sum(-1), 1.0, atol=1e-12)


def test_block_mass_uniform_case_and_supplied_lse():
    """Q = 0 => every key gets 1/N, so mass[I, J] = |J| / N exactly; an LSE taken from the (pinned)
    attention oracle's dense run gives the same masses as the internal one."""
    rng = np.random.default_rng(21)
    N, D = 45, 8
    Q, K, V = (rand_bits(rng, (1, 1, N, D)) for _ in range(3))
    M0 = orc.block_mass_exact(np.zeros_like(Q[0, 0]), K[0, 0], N, 16, 8, 0.3)
    sizes = np.minimum(8, N - np.arange(6) * 8) / N
    np.testing.assert_allclose(M0, np.tile(sizes, (3, 1)), atol=1e-12)
    ones = np.ones((1, 1, 3, 6), dtype=np.uint8)
    _, L = orc.attention_full(Q, K, V, N, 16, 8, 0.3, ones)
    np.testing.assert_allclose(orc.block_mass_exact(Q[0, 0], K[0, 0], N, 16, 8, 0.3, lse=L[0, 0]),
                               orc.block_mass_exact(Q[0, 0], K[0, 0], N, 16, 8, 0.3), atol=1e-12)


def test_select_by_mass_is_smallest_covering_descending_prefix():
    rng = np.random.default_rng(22)
    for trial in range(60):
        n = int(rng.integers(2, 40))
        m = rng.random(n).astype(np.float32) ** 4
        m[rng.random(n) < 0.2] = m[0]                     # ties
        forced = rng.random(n) < 0.15
        tau = float(rng.choice([0.5, 0.9, 0.99]))
        keep, theta = orc.select_by_mass(m, forced, tau)
        p = m.astype(np.float64) / m.astype(np.float64).sum()
        t32 = float(np.float32(tau))
        assert keep[forced].all() and p[keep].sum() >= t32 - 1e-12
        adm = keep & ~forced
        if adm.any():
            weakest = min(np.nonzero(adm)[0], key=lambda j: (float(m[j]), -j))
            assert p[keep].sum() - p[weakest] < t32            # minimal
            assert theta == m[weakest]
            if (~keep).any():
                assert m[adm].min() >= m[~keep].max()          # a descending prefix
            # equal masses: lower index first
            eq = [j for j in range(n) if not forced[j] and m[j] == m[weakest]]
            kept_eq = [j for j in eq if keep[j]]
            assert kept_eq == eq[:len(kept_eq)]
        else:
            assert p[forced].sum() >= t32


def test_exact_rule_agrees_with_cummass_rule_on_log_masses():
    """select_cummass on scores = ln(mass) is the same rule (softmax of ln m = m / sum m)."""
    rng = np.random.default_rng(23)
    m = (rng.random(24) ** 3 + 1e-3).astype(np.float32)
    forced = np.zeros(24, dtype=bool); forced[3] = True
    k1, _ = orc.select_by_mass(m, forced, 0.8)
    k2, _ = orc.select_cummass(np.log(m.astype(np.float64)).astype(np.float32), forced, 0.8)
    np.testing.assert_array_equal(k1, k2)


def test_build_connectivity_exact_and_estimator_recall_is_reported():
    """Exact rule on a structured slice; the recall of the pooled estimator against it is only reported."""
    w = wl.shrunk(wl.get("wan1p3b_480p"), H=1, T=4, Hg=16, Wg=16)
    Q, K, _ = wl.gen_qkv(w, "history")
    mask, masses, theta, F = orc.build_connectivity_exact(Q, K, w.N, 0, w.T, w.Hg, w.Wg, 128, 128, w.scale, mass=0.9)
    np.testing.assert_allclose(masses.sum(-1), 1.0, atol=1e-5)
    kept = (masses * (mask != 0)).sum(-1)
    assert (kept >= 0.9 - 1e-6).all()
    est, _, _, _ = orc.build_connectivity(Q, K, w.N, 0, w.T, w.Hg, w.Wg, 128, 128, w.scale,
                                          orc.MODE_CUMMASS, 0.25, 0.9, -1, 0, 1)
    recall = float(((est != 0) & (mask != 0)).sum() / max(1, (mask != 0).sum()))
    print(f"pooled estimator recall of the exact 0.9-mass blocks: {recall:.3f}")
    assert 0.0 <= recall <= 1.0
