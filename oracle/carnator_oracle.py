"""CPU oracle for the block-sparse attention path and its connectivity builder.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path imports this module; it
is called by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark.  It shares no code with the CUDA path: plain numpy, fp64 unless a
step says otherwise, no tiling, no online softmax.

What it computes follows the paper's description of historical
sparse-connectivity reuse (Section 3.3, "Historical Sparse-Connectivity Reuse"
and "Joint Reuse in Intermediate Layers"; Appendix "Reuse-Scope Implementation
Details"; Algorithm 1, the last two lines of the denoising loop):

* attention: the target's own Q, K, V; a query attends exactly to the keys
  whose (query block, key block) pair is present in the historical block mask,
  or to every key when its query block is flagged target-specific
  ("recompute").  The result is ordinary softmax attention restricted to that
  key set, so the oracle is that definition written out.
* connectivity builder: self-attention is partitioned into query x key blocks
  and, per head and query block, the smallest set of key blocks that covers a
  fixed fraction of the attention mass is kept (Appendix "Reuse-Scope
  Implementation Details").  The graded form estimates block mass from
  block-pooled Q.K^T scores and selects per row by top-k or by cumulative
  softmax mass; it is an estimator plus a selection rule, so the oracle takes
  the steps in order.

Pin status (tests/test_oracle_*.py):
  attention_rows / attention_full ... pinned (brute force, closed forms, invariants, hand-worked fixture)
  pooled_scores ..................... pinned (bilinearity identity vs. per-token brute force)
  forced_blocks ..................... pinned (per-token brute force)
  select_topk / select_cummass ...... pinned (stable sort, counts, order and minimality invariants)
  block_mass_exact / select_by_mass / build_connectivity_exact ... pinned (brute force, closed form, invariants)
  build_regions / fuse_latents / region_block_flags / attention_region_rows ... pinned (definitions by hand, closed forms)
  seed_expansion ... pinned (dense softmax matrix by brute force, invariants)
  clopper_pearson_upper ... pinned (value printed in the paper, closed form for u = 0); delta_e00 / shape / size ... pinned (closed forms, invariants)
  fidelity of the pooled estimator to the true block attention mass: PARITY UNPINNED
  (the paper prints no mask, density or recall figure; it can only be reported, see tests).
"""
from __future__ import annotations

import math
from typing import Iterable, List, Optional, Sequence, Tuple

import numpy as np

MODE_TOPK = 0
MODE_CUMMASS = 1


def _widen(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64, exactly."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# ==========================================================================
# Attention under a block mask  (Section 3.3, Historical Sparse-Connectivity Reuse)
# ==========================================================================
def allowed_key_blocks(mask_row: np.ndarray, recompute_flag: int) -> np.ndarray:
    """Key blocks a query block may attend to: every block if the query block is
    flagged for recomputation, else the non-zero entries of its mask row."""
    nkb = mask_row.shape[0]
    if recompute_flag:
        return np.arange(nkb)
    return np.nonzero(mask_row)[0]


def attention_rows(Qb: np.ndarray, Kb: np.ndarray, Vb: np.ndarray, N: int,
                   block_q: int, block_k: int, scale: float,
                   mask: np.ndarray, recompute: Optional[np.ndarray],
                   rows: Sequence[Tuple[int, int, int]]):
    """Masked softmax attention for the listed query blocks.

    Qb, Kb, Vb : uint16 bf16 bits [B, H, >=N, D]
    mask       : uint8 [B, H, nqb, nkb], non-zero = evaluate the block pair
    recompute  : uint8 [B, nqb] or None, non-zero = the query block sees every key
    rows       : (b, h, I) triples

    Returns O [len(rows), block_q, D] and LSE [len(rows), block_q] in fp64; entries
    of query tokens >= N are NaN.  A query with an empty key set gets O = 0,
    LSE = -inf.  LSE is the natural log of the sum of exp(scaled scores).
    """
    D = Qb.shape[-1]
    O = np.full((len(rows), block_q, D), np.nan)
    LSE = np.full((len(rows), block_q), np.nan)
    cache_key = None
    K64 = V64 = None
    for r, (b, h, I) in enumerate(rows):
        if cache_key != (b, h):
            K64 = _widen(Kb[b, h, :N])
            V64 = _widen(Vb[b, h, :N])
            cache_key = (b, h)
        i0, i1 = I * block_q, min(N, (I + 1) * block_q)
        if i0 >= N:
            continue
        q = _widen(Qb[b, h, i0:i1])
        flag = int(recompute[b, I]) if recompute is not None else 0
        blocks = allowed_key_blocks(mask[b, h, I], flag)
        cols = [np.arange(J * block_k, min(N, (J + 1) * block_k)) for J in blocks]
        cols = np.concatenate(cols) if len(cols) else np.zeros((0,), dtype=np.int64)
        if cols.size == 0:
            O[r, : i1 - i0] = 0.0
            LSE[r, : i1 - i0] = -np.inf
            continue
        s = scale * (q @ K64[cols].T)                 # s_ij for j in the allowed set
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        l = p.sum(axis=1, keepdims=True)
        O[r, : i1 - i0] = (p @ V64[cols]) / l
        LSE[r, : i1 - i0] = (m + np.log(l))[:, 0]
    return O, LSE


def attention_full(Qb, Kb, Vb, N, block_q, block_k, scale, mask, recompute=None):
    """All query blocks of all heads: O [B, H, N, D], LSE [B, H, N] in fp64."""
    B, H = Qb.shape[0], Qb.shape[1]
    D = Qb.shape[-1]
    nqb = -(-N // block_q)
    rows = [(b, h, I) for b in range(B) for h in range(H) for I in range(nqb)]
    Or, Lr = attention_rows(Qb, Kb, Vb, N, block_q, block_k, scale, mask, recompute, rows)
    O = Or.reshape(B, H, nqb * block_q, D)[:, :, :N]
    L = Lr.reshape(B, H, nqb * block_q)[:, :, :N]
    return O, L


def dense_bruteforce(Qb, Kb, Vb, N, block_q, block_k, scale, mask, recompute=None):
    """Second, independent statement of the same definition, for tiny inputs only.

    Materialises the N x N score matrix of each head with -inf at every
    disallowed (query, key) pair and evaluates softmax one query at a time with
    Python scalars.  Used only to check attention_rows / attention_full.
    """
    B, H = Qb.shape[0], Qb.shape[1]
    D = Qb.shape[-1]
    O = np.zeros((B, H, N, D))
    LSE = np.zeros((B, H, N))
    for b in range(B):
        for h in range(H):
            q = _widen(Qb[b, h, :N])
            k = _widen(Kb[b, h, :N])
            v = _widen(Vb[b, h, :N])
            S = np.full((N, N), -np.inf)
            for i in range(N):
                I = i // block_q
                dense = recompute is not None and recompute[b, I] != 0
                for j in range(N):
                    if dense or mask[b, h, I, j // block_k] != 0:
                        acc = 0.0
                        for d in range(D):
                            acc += q[i, d] * k[j, d]
                        S[i, j] = scale * acc
            for i in range(N):
                mx = max(S[i])
                if mx == -np.inf:
                    LSE[b, h, i] = -np.inf
                    continue
                den = 0.0
                num = np.zeros(D)
                for j in range(N):
                    if S[i, j] != -np.inf:
                        e = math.exp(S[i, j] - mx)
                        den += e
                        num += e * v[j]
                O[b, h, i] = num / den
                LSE[b, h, i] = mx + math.log(den)
    return O, LSE


# ==========================================================================
# Connectivity builder  (Appendix "Reuse-Scope Implementation Details")
# ==========================================================================
def pooled_means(Xb_head: np.ndarray, N: int, block: int) -> np.ndarray:
    """Step 1: mean of each block's VALID token rows, fp64 accumulate -> fp32.  [nb, D] float32."""
    nb = -(-N // block)
    X = _widen(Xb_head[:N])
    out = np.zeros((nb, X.shape[1]), dtype=np.float32)
    for I in range(nb):
        seg = X[I * block: min(N, (I + 1) * block)]
        out[I] = (seg.sum(axis=0) / seg.shape[0]).astype(np.float32)
    return out


def pooled_scores(Qb_head, Kb_head, N, block_q, block_k, scale) -> np.ndarray:
    """Step 2: S~[I, J] = fp32(scale * <q_bar_I, k_bar_J>), fp64 accumulate.  This fp32
    value is 'the pooled score' that selection and the tolerance band refer to."""
    qbar = pooled_means(Qb_head, N, block_q).astype(np.float64)
    kbar = pooled_means(Kb_head, N, block_k).astype(np.float64)
    return (np.float64(np.float32(scale)) * (qbar @ kbar.T)).astype(np.float32)


def forced_blocks(N, n_text, T, Hg, Wg, block_q, block_k, window_frames, text_dense) -> np.ndarray:
    """Step 3: bool [nqb, nkb], blocks kept regardless of score.

    text_dense: a query block holding a text token keeps every key block, and every
    key block holding a text token is kept by every query block.
    window_frames = r >= 0: a query block whose video tokens span frames f_lo..f_hi
    keeps every key block holding a video token of frames [f_lo - r, f_hi + r].
    Token order: text first, then video flattened frame-major.
    """
    nqb, nkb = -(-N // block_q), -(-N // block_k)
    hw = Hg * Wg
    F = np.zeros((nqb, nkb), dtype=bool)

    def frames_of(block, I):
        lo, hi = I * block, min(N, (I + 1) * block) - 1
        lo = max(lo, n_text)
        if hi < lo:
            return None
        return (lo - n_text) // hw, (hi - n_text) // hw

    kf = [frames_of(block_k, J) for J in range(nkb)]
    for I in range(nqb):
        if text_dense and n_text > 0 and I * block_q < n_text:
            F[I, :] = True
            continue
        if text_dense and n_text > 0:
            for J in range(nkb):
                if J * block_k < n_text:
                    F[I, J] = True
        if window_frames >= 0:
            qf = frames_of(block_q, I)
            if qf is not None:
                lo = max(0, qf[0] - window_frames)
                hi = min(T - 1, qf[1] + window_frames)
                for J in range(nkb):
                    if kf[J] is not None and kf[J][0] <= hi and kf[J][1] >= lo:
                        F[I, J] = True
    return F


def topk_count(keep_ratio: float, n_candidates: int) -> int:
    """k = ceil(ratio * n - 1e-6) clamped to [1, n] (0 when there is no candidate).
    The ratio is taken at fp32 precision, as it travels through the C struct."""
    if n_candidates <= 0:
        return 0
    k = math.ceil(float(np.float32(keep_ratio)) * n_candidates - 1e-6)
    return max(1, min(n_candidates, k))


def _descending_stable(scores: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """idx reordered by score descending; equal scores keep ascending block index."""
    order = np.argsort(-scores[idx].astype(np.float64), kind="stable")
    return idx[order]


def select_topk(scores_row: np.ndarray, forced_row: np.ndarray, keep_ratio: float,
                count_includes_forced: int):
    """Step 4.  Returns (keep bool[nkb], theta) with theta the score of the last block
    admitted by score (NaN if none was)."""
    nkb = scores_row.shape[0]
    keep = forced_row.copy()
    free = np.nonzero(~forced_row)[0]
    if count_includes_forced:
        k = topk_count(keep_ratio, nkb)
        n_admit = max(0, k - int(forced_row.sum()))
    else:
        n_admit = topk_count(keep_ratio, free.size)
    n_admit = min(n_admit, free.size)
    theta = np.float32(np.nan)
    if n_admit > 0:
        ranked = _descending_stable(scores_row, free)
        keep[ranked[:n_admit]] = True
        theta = scores_row[ranked[n_admit - 1]]
    return keep, theta


def select_cummass(scores_row: np.ndarray, forced_row: np.ndarray, mass: float):
    """Step 5.  p = softmax over all key blocks of the pooled scores (fp64); non-forced
    blocks are admitted in descending score order until the kept mass (forced blocks
    included) reaches ``mass`` -- the smallest descending prefix that covers it."""
    s = scores_row.astype(np.float64)
    p = np.exp(s - s.max())
    p = p / p.sum()
    keep = forced_row.copy()
    free = np.nonzero(~forced_row)[0]
    ranked = _descending_stable(scores_row, free)
    target = float(np.float32(mass))
    running = float(p[forced_row].sum())
    theta = np.float32(np.nan)
    for J in ranked:
        if running >= target:
            break
        keep[J] = True
        running += p[J]
        theta = scores_row[J]
    return keep, theta


def build_connectivity(Qb, Kb, N, n_text, T, Hg, Wg, block_q, block_k, scale,
                       mode=MODE_TOPK, keep_ratio=0.25, mass=0.9, window_frames=-1,
                       text_dense=0, count_includes_forced=1,
                       heads: Optional[Iterable[Tuple[int, int]]] = None):
    """Steps 1-6 for every (or the listed) head.

    Returns mask uint8 [B, H, nqb, nkb], scores float32 [B, H, nqb, nkb],
    theta float32 [B, H, nqb] (NaN where no block was admitted by score) and the
    forced-block table bool [nqb, nkb].  Heads not listed stay zero.
    """
    B, H = Qb.shape[0], Qb.shape[1]
    nqb, nkb = -(-N // block_q), -(-N // block_k)
    F = forced_blocks(N, n_text, T, Hg, Wg, block_q, block_k, window_frames, text_dense)
    mask = np.zeros((B, H, nqb, nkb), dtype=np.uint8)
    scores = np.zeros((B, H, nqb, nkb), dtype=np.float32)
    theta = np.full((B, H, nqb), np.nan, dtype=np.float32)
    todo = list(heads) if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    for (b, h) in todo:
        S = pooled_scores(Qb[b, h], Kb[b, h], N, block_q, block_k, scale)
        scores[b, h] = S
        for I in range(nqb):
            if mode == MODE_TOPK:
                keep, th = select_topk(S[I], F[I], keep_ratio, count_includes_forced)
            elif mode == MODE_CUMMASS:
                keep, th = select_cummass(S[I], F[I], mass)
            else:
                raise ValueError("unknown selection mode")
            mask[b, h, I] = keep
            theta[b, h, I] = th
    return mask, scores, theta, F


def block_mass_exact(Qb_head, Kb_head, N, block_q, block_k, scale, lse: Optional[np.ndarray] = None) -> np.ndarray:
    """The paper's literal quantity (Appendix "Reuse-Scope Implementation Details": the attention
    mass a query block sends to each key block): mass[I, J] = (1/|I|) * sum_{i in I} sum_{j in J}
    exp(s_ij - LSE_i), LSE_i the log-sum-exp of query i over ALL keys.  [nqb, nkb] fp64; each row
    sums to 1.  ``lse`` (natural log, [N]) may be supplied -- e.g. the LSE a dense attention run
    returned; otherwise it is computed here from the same scores."""
    q = _widen(Qb_head[:N])
    k = _widen(Kb_head[:N])
    nqb, nkb = -(-N // block_q), -(-N // block_k)
    starts = np.arange(nkb) * block_k
    out = np.zeros((nqb, nkb))
    for I in range(nqb):
        i0, i1 = I * block_q, min(N, (I + 1) * block_q)
        s = scale * (q[i0:i1] @ k.T)
        l = lse[i0:i1, None] if lse is not None else np.logaddexp.reduce(s, axis=1, keepdims=True)
        p = np.exp(s - l)
        out[I] = np.add.reduceat(p, starts, axis=1).sum(axis=0) / (i1 - i0)
    return out


def select_by_mass(mass_row: np.ndarray, forced_row: np.ndarray, target: float):
    """Smallest descending prefix of the non-forced key blocks whose mass, together with the forced
    blocks', reaches ``target`` of the row's total (ties: lower block index first).  Returns
    (keep bool[nkb], theta) with theta the mass of the last admitted block (NaN if none)."""
    m = mass_row.astype(np.float64)
    p = m / m.sum()
    keep = forced_row.copy()
    free = np.nonzero(~forced_row)[0]
    ranked = _descending_stable(mass_row, free)
    tgt = float(np.float32(target))
    running = float(p[forced_row].sum())
    theta = np.float32(np.nan)
    for J in ranked:
        if running >= tgt:
            break
        keep[J] = True
        running += p[J]
        theta = mass_row[J]
    return keep, theta


def build_connectivity_exact(Qb, Kb, N, n_text, T, Hg, Wg, block_q, block_k, scale, mass=0.9,
                             window_frames=-1, text_dense=0, lse: Optional[np.ndarray] = None,
                             heads: Optional[Iterable[Tuple[int, int]]] = None):
    """The paper's rule on the exact block masses: per head and query block keep the smallest set of
    key blocks covering ``mass`` of the attention mass (always-kept blocks included).  ``lse`` is
    [B, H, N] or None.  Returns mask uint8, masses float32 [B,H,nqb,nkb], theta, forced table."""
    B, H = Qb.shape[0], Qb.shape[1]
    nqb, nkb = -(-N // block_q), -(-N // block_k)
    F = forced_blocks(N, n_text, T, Hg, Wg, block_q, block_k, window_frames, text_dense)
    mask = np.zeros((B, H, nqb, nkb), dtype=np.uint8)
    masses = np.zeros((B, H, nqb, nkb), dtype=np.float32)
    theta = np.full((B, H, nqb), np.nan, dtype=np.float32)
    todo = list(heads) if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    for (b, h) in todo:
        M = block_mass_exact(Qb[b, h], Kb[b, h], N, block_q, block_k, scale,
                             None if lse is None else lse[b, h]).astype(np.float32)
        masses[b, h] = M
        for I in range(nqb):
            keep, th = select_by_mass(M[I], F[I], mass)
            mask[b, h, I] = keep
            theta[b, h, I] = th
    return mask, masses, theta, F


# ==========================================================================
# Reuse regions, latent fusion, region-restricted connectivity
# (Section 3.3 "Region-Guided Latent Reuse" and "Joint Reuse in Intermediate Layers";
#  Appendix "Reuse-Scope Implementation Details")
# ==========================================================================
def chebyshev_distance_per_frame(src: np.ndarray) -> np.ndarray:
    """For every token of a [T, H, W] grid, the Chebyshev distance (max of row and column offsets)
    to the nearest True token of ``src`` in the SAME frame; a large number (T*H*W) where the frame
    holds none.  Plain search, written for small grids."""
    T, H, W = src.shape
    big = T * H * W
    out = np.full((T, H, W), big, dtype=np.int64)
    for t in range(T):
        ys, xs = np.nonzero(src[t])
        if len(ys) == 0:
            continue
        for y in range(H):
            for x in range(W):
                out[t, y, x] = np.maximum(np.abs(ys - y), np.abs(xs - x)).min()
    return out


def dilate_per_frame(src: np.ndarray, radius: int) -> np.ndarray:
    """Dilation by ``radius`` tokens on the H x W grid of each latent frame (square neighbourhood,
    i.e. every token within Chebyshev distance ``radius`` of the region; no wrap-around)."""
    return chebyshev_distance_per_frame(src) <= radius


def smoothstep(x):
    return 3.0 * x * x - 2.0 * x * x * x


def build_regions(evidence: np.ndarray, r_active: int = 2, r_context: int = 3):
    """Active region = evidence dilated by r_active, context region = active dilated by a further
    r_context (per latent frame).  Blend weight W: 1 on the evidence region, 1 - smoothstep(d_hat)
    on the transition band active minus evidence, 0 outside the active region, where d_hat is the
    Chebyshev distance to the evidence region divided by the largest such distance attained in the
    band (taken over the whole band).  Returns (active bool, context bool, W float64), all [T, H, W]."""
    ev = evidence != 0
    d = chebyshev_distance_per_frame(ev)
    active = d <= r_active
    context = chebyshev_distance_per_frame(active) <= r_context
    band = active & ~ev
    W = np.zeros(ev.shape, dtype=np.float64)
    W[ev] = 1.0
    if band.any():
        dmax = float(d[band].max())
        W[band] = 1.0 - smoothstep(d[band] / dmax)
    return active, context, W


def fuse_latents(z_target: np.ndarray, z_hist: np.ndarray, W: np.ndarray) -> np.ndarray:
    """z = W * z_target + (1 - W) * z_hist, W broadcast over the leading (channel) axes; fp64."""
    zt = np.asarray(z_target, dtype=np.float64)
    zh = np.asarray(z_hist, dtype=np.float64)
    return W * zt + (1.0 - W) * zh


def region_block_flags(region: np.ndarray, n_text: int, block: int, text_value: int = 1) -> np.ndarray:
    """uint8 per block of the token order (text first, then the grid flattened frame-major): 1 if the
    block holds a token of the region.  Text tokens count as members when text_value is 1."""
    flat = np.concatenate([np.full(n_text, bool(text_value)), (region != 0).ravel()])
    nb = -(-flat.size // block)
    out = np.zeros(nb, dtype=np.uint8)
    for I in range(nb):
        out[I] = 1 if flat[I * block:(I + 1) * block].any() else 0
    return out


def attention_region_rows(Qb, Kb, Vb, N, block_q, block_k, scale, mask, active_q, context_k, rows):
    """Middle-layer form: the historical connectivity restricted to active query blocks and context key
    blocks (mask AND active x context); query blocks that are not active are not computed at all (their
    rows come back NaN: the caller keeps the cached values).  active_q [B, nqb], context_k [B, nkb]."""
    B = mask.shape[0]
    eff = mask.copy()
    for b in range(B):
        eff[b] = mask[b] * (context_k[b] != 0)[None, None, :]
    O, L = attention_rows(Qb, Kb, Vb, N, block_q, block_k, scale, eff, None, rows)
    for r, (b, h, I) in enumerate(rows):
        if active_q[b, I] == 0:
            O[r] = np.nan
            L[r] = np.nan
    return O, L


# ==========================================================================
# Seeded self-attention expansion (Section 3.2; Appendix "Evidence Region Construction")
# ==========================================================================
def seed_expansion(Qb, Kb, N, scale, seeds_pos, seeds_neg, lse: Optional[np.ndarray] = None,
                   heads=None, rows: Optional[np.ndarray] = None):
    """S_i = mean_h [ max_{u in I+} A_h[i,u] - max_{u in I-} A_h[i,u] ] with A the dense self-attention
    weights (softmax over all N keys).  Returns (contrast [B, N], per_head [B, H, N]) in fp64.  ``lse``
    [B, H, N] may be supplied; otherwise the softmax normaliser is computed here.  An empty seed set
    contributes 0.  With ``heads`` (a list of (b, h)) and / or ``rows`` (query token indices) only those
    entries of per_head are computed (the others stay 0, and the contrast is then not meaningful): the
    same arithmetic, for sampled checks of layers too large to do in full."""
    B, H = Qb.shape[0], Qb.shape[1]
    per_head = np.zeros((B, H, N))
    sp = np.asarray(seeds_pos, dtype=np.int64)
    sn = np.asarray(seeds_neg, dtype=np.int64)
    sel = np.arange(N) if rows is None else np.asarray(rows, dtype=np.int64)
    todo = [(b, h) for b in range(B) for h in range(H)] if heads is None else list(heads)
    for (b, h) in todo:
        q, k = _widen(Qb[b, h, :N])[sel], _widen(Kb[b, h, :N])
        if lse is None:
            l = np.zeros(len(sel))
            for i0 in range(0, len(sel), 1024):
                l[i0:i0 + 1024] = np.logaddexp.reduce(scale * (q[i0:i0 + 1024] @ k.T), axis=1)
        else:
            l = lse[b, h][sel]
        pos = np.exp(scale * (q @ k[sp].T) - l[:, None]).max(axis=1) if sp.size else 0.0
        neg = np.exp(scale * (q @ k[sn].T) - l[:, None]).max(axis=1) if sn.size else 0.0
        per_head[b, h, sel] = pos - neg
    return per_head.mean(axis=1), per_head


# ==========================================================================
# Compatibility scalars and the risk certificate
# (Section 3.2; Appendix "Risk-Aware Compatibility Decision")
# ==========================================================================
def delta_e00(lab1, lab2) -> float:
    """CIEDE2000 colour difference (k_L = k_C = k_H = 1), vectorised-formula form in numpy."""
    L1, a1, b1 = (float(v) for v in lab1)
    L2, a2, b2 = (float(v) for v in lab2)
    C1, C2 = np.hypot(a1, b1), np.hypot(a2, b2)
    Cbar = (C1 + C2) / 2
    G = 0.5 * (1 - np.sqrt(Cbar ** 7 / (Cbar ** 7 + 25.0 ** 7)))
    a1p, a2p = (1 + G) * a1, (1 + G) * a2
    C1p, C2p = np.hypot(a1p, b1), np.hypot(a2p, b2)
    h1p = np.degrees(np.arctan2(b1, a1p)) % 360 if (a1p or b1) else 0.0
    h2p = np.degrees(np.arctan2(b2, a2p)) % 360 if (a2p or b2) else 0.0
    dLp, dCp = L2 - L1, C2p - C1p
    if C1p * C2p == 0:
        dhp = 0.0
    else:
        dhp = h2p - h1p
        dhp = dhp - 360 if dhp > 180 else (dhp + 360 if dhp < -180 else dhp)
    dHp = 2 * np.sqrt(C1p * C2p) * np.sin(np.radians(dhp / 2))
    Lbar, Cbarp = (L1 + L2) / 2, (C1p + C2p) / 2
    if C1p * C2p == 0:
        hbar = h1p + h2p
    elif abs(h1p - h2p) <= 180:
        hbar = (h1p + h2p) / 2
    else:
        hbar = (h1p + h2p + 360) / 2 if h1p + h2p < 360 else (h1p + h2p - 360) / 2
    T = (1 - 0.17 * np.cos(np.radians(hbar - 30)) + 0.24 * np.cos(np.radians(2 * hbar))
         + 0.32 * np.cos(np.radians(3 * hbar + 6)) - 0.20 * np.cos(np.radians(4 * hbar - 63)))
    dtheta = 30 * np.exp(-(((hbar - 275) / 25) ** 2))
    RC = 2 * np.sqrt(Cbarp ** 7 / (Cbarp ** 7 + 25.0 ** 7))
    SL = 1 + 0.015 * (Lbar - 50) ** 2 / np.sqrt(20 + (Lbar - 50) ** 2)
    SC, SH = 1 + 0.045 * Cbarp, 1 + 0.015 * Cbarp * T
    RT = -np.sin(np.radians(2 * dtheta)) * RC
    return float(np.sqrt((dLp / SL) ** 2 + (dCp / SC) ** 2 + (dHp / SH) ** 2 + RT * (dCp / SC) * (dHp / SH)))


def context_discrepancy(labs_q, labs_j) -> float:
    """d_context (Section 3.2, discrepancy vector): the largest CIEDE2000 difference between the target's and the
    historical request's mean CIELAB colours over the shared nouns; 0 when no noun is shared.
    labs_q[o], labs_j[o]: the (L*, a*, b*) of shared noun o in the two requests."""
    d = 0.0
    for cq, cj in zip(labs_q, labs_j):
        d = max(d, delta_e00(cq, cj))
    return d


def bbox_normalized(m: np.ndarray, res: int) -> np.ndarray:
    """Crop a binary indicator to its tight support box and resample to res x res (nearest, cell centres)."""
    ys, xs = np.nonzero(m)
    box = m[ys.min():ys.max() + 1, xs.min():xs.max() + 1]
    r = np.minimum(box.shape[0] - 1, ((np.arange(res) + 0.5) * box.shape[0] / res).astype(int))
    c = np.minimum(box.shape[1] - 1, ((np.arange(res) + 0.5) * box.shape[1] / res).astype(int))
    return (box[np.ix_(r, c)] != 0)


def shape_discrepancy(m_q: np.ndarray, m_j: np.ndarray, res: int = 32) -> float:
    a, b = bbox_normalized(m_q, res), bbox_normalized(m_j, res)
    return 1.0 - 2.0 * float((a & b).sum()) / float(a.sum() + b.sum())


def size_discrepancy(area_q: float, area_j: float) -> float:
    return abs(math.log(area_q / area_j))


def compatibility_gate(d, tau, applicable=None) -> int:
    return int(all((dk <= tk) for k, (dk, tk) in enumerate(zip(d, tau)) if applicable is None or applicable[k]))


def clopper_pearson_upper(u: int, n: int, alpha: float) -> float:
    """One-sided upper limit: the (1 - alpha) quantile of Beta(u + 1, n - u) (library routine)."""
    from scipy.stats import beta
    if u >= n:
        return 1.0
    return float(beta.ppf(1.0 - alpha, u + 1, n - u))


# ==========================================================================
# counting helpers used by tests and the benchmark
# ==========================================================================
def computed_tile_flops(N, D, block_q, block_k, mask, recompute=None) -> float:
    """4 * rows_valid * cols_valid * D summed over evaluated block pairs (all heads)."""
    B, H, nqb, nkb = mask.shape
    rq = np.minimum(block_q, N - np.arange(nqb) * block_q).astype(np.float64)
    ck = np.minimum(block_k, N - np.arange(nkb) * block_k).astype(np.float64)
    total = 0.0
    for b in range(B):
        eff = mask[b] != 0
        if recompute is not None:
            eff = eff | (recompute[b] != 0)[None, :, None]
        total += 4.0 * D * float(np.einsum("hij,i,j->", eff.astype(np.float64), rq, ck))
    return total
