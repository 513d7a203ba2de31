"""Shared helpers for the tests: random bf16 bit tensors and tolerance checks."""
import numpy as np

from paper_2609_32420_b200 import workloads as wl


def rand_bits(rng, shape, scale=1.0):
    return wl.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def widen(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def record(kind, what, **values):
    """Append one line of measured parity errors to the file named by CARNATOR_PARITY_LOG (if set)."""
    import json
    import os
    path = os.environ.get("CARNATOR_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps({"kind": kind, "case": what, **values}) + "\n")


# tolerances the GPU path must meet against the oracle
O_MAX_ABS = 2e-2
O_MEAN_ABS = 2e-3
LSE_REL = 1e-3
SCORE_BAND = 1e-4


def check_attention(O_gpu, LSE_gpu, O_ref, LSE_ref, what=""):
    """O: max abs <= 2e-2 and mean abs <= 2e-3; LSE: |d| <= 1e-3 * max(|ref|, 1); -inf must match exactly."""
    O_gpu = np.asarray(O_gpu, dtype=np.float64)
    O_ref = np.asarray(O_ref, dtype=np.float64)
    ok = ~np.isnan(O_ref)
    assert np.isfinite(O_gpu[ok]).all(), f"{what}: non-finite O"
    err = np.abs(O_gpu[ok] - O_ref[ok])
    assert err.max(initial=0.0) <= O_MAX_ABS, f"{what}: O max abs {err.max()}"
    assert (err.mean() if err.size else 0.0) <= O_MEAN_ABS, f"{what}: O mean abs {err.mean()}"
    L_gpu = np.asarray(LSE_gpu, dtype=np.float64)
    L_ref = np.asarray(LSE_ref, dtype=np.float64)
    okl = ~np.isnan(L_ref)
    ninf = okl & np.isneginf(L_ref)
    assert np.isneginf(L_gpu[ninf]).all(), f"{what}: LSE of an empty row must be -inf"
    fin = okl & ~ninf
    rel = np.abs(L_gpu[fin] - L_ref[fin]) / np.maximum(np.abs(L_ref[fin]), 1.0)
    assert rel.max(initial=0.0) <= LSE_REL, f"{what}: LSE rel {rel.max()}"
    out = float(err.max(initial=0.0)), float(err.mean() if err.size else 0.0), float(rel.max(initial=0.0))
    record("attention", what, o_max_abs=out[0], o_mean_abs=out[1], lse_rel=out[2], n_values=int(err.size))
    return out


def check_mask(mask_gpu, mask_ref, scores_ref, theta_ref, forced, topk_mode=True, what=""):
    """Bit-exact except blocks whose oracle pooled score lies within 1e-4 of the row's
    selection threshold; forced blocks are never excusable; in top-k mode the row count must match."""
    mask_gpu = np.asarray(mask_gpu) != 0
    mask_ref = np.asarray(mask_ref) != 0
    diff = mask_gpu != mask_ref
    n_diff = int(diff.sum())
    record("mask", what, mismatches=n_diff, blocks=int(mask_ref.size), density=float(mask_ref.mean()))
    if n_diff == 0:
        return 0
    B, H, nqb, nkb = mask_ref.shape
    b, h, I, J = np.nonzero(diff)
    assert not forced[I, J].any(), f"{what}: mismatch on a forced block"
    th = theta_ref[b, h, I]
    assert not np.isnan(th).any(), f"{what}: mismatch in a row with no score-admitted block"
    near = np.abs(scores_ref[b, h, I, J].astype(np.float64) - th.astype(np.float64)) <= SCORE_BAND
    assert near.all(), f"{what}: {int((~near).sum())} mask mismatches outside the 1e-4 band"
    if topk_mode:
        assert (mask_gpu.sum(-1) == mask_ref.sum(-1)).all(), f"{what}: row counts differ"
    return n_diff
