"""Comparators used by the parity tests (CPU-only code; no CUDA, no oracle arithmetic)."""
from __future__ import annotations

import numpy as np

# Acceptance tolerances of the attention outputs (bf16 inputs, fp32 accumulate on the GPU,
# fp64 oracle): max absolute error and per-row relative L2 error.
MAX_ABS = 1e-2
ROW_REL_L2 = 5e-3
LSE_ABS = 1e-3
# Routing may differ from the oracle only inside this relative window around the k-th score.
NEAR_TIE = 1e-3


def check_routing(gpu_idx: np.ndarray, ref_idx: np.ndarray, ref_scores_all: np.ndarray):
    """Bit-exact comparison of the selected chunk sets with the near-tie rule.

    A row may differ from the oracle only if the oracle's k-th / (k+1)-th score gap is within
    NEAR_TIE * |k-th score|, and only by exchanging chunks whose oracle scores lie within that
    window of the k-th score.  Returns the number of excused rows; raises on any other mismatch.
    """
    B, Hkv, k = ref_idx.shape
    C = ref_scores_all.shape[-1]
    assert gpu_idx.shape == ref_idx.shape
    excused = 0
    for b in range(B):
        for h in range(Hkv):
            g, r = gpu_idx[b, h], ref_idx[b, h]
            assert np.all(np.diff(g) > 0), f"row ({b},{h}): GPU indices not strictly ascending: {g}"
            assert g.min() >= 0 and g.max() < C
            if np.array_equal(g, r):
                continue
            sc = ref_scores_all[b, h]
            order = np.argsort(-sc, kind="stable")
            s_k = sc[order[k - 1]]
            gap = s_k - sc[order[k]] if k < C else np.inf
            window = NEAR_TIE * abs(s_k)
            assert gap <= window, (
                f"row ({b},{h}): routing differs but the k/(k+1) gap {gap:.3e} exceeds the "
                f"near-tie window {window:.3e}: gpu {g} oracle {r}")
            diff = np.setxor1d(g, r)
            assert np.all(np.abs(sc[diff] - s_k) <= window), (
                f"row ({b},{h}): exchanged chunks {diff} are not near ties of the k-th score")
            excused += 1
    return excused


def check_attention(gpu, ref, what: str, max_abs: float = MAX_ABS, row_rel: float = ROW_REL_L2):
    """gpu, ref: [..., D] arrays (ref in float64).  Checks max-abs and per-row relative L2."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, f"{what}: shape {gpu.shape} vs {ref.shape}"
    assert np.all(np.isfinite(gpu)), f"{what}: non-finite values in the GPU result"
    err = np.abs(gpu - ref)
    worst = err.max() if err.size else 0.0
    assert worst <= max_abs, f"{what}: max abs error {worst:.3e} > {max_abs}"
    num = np.sqrt((err ** 2).sum(axis=-1))
    den = np.sqrt((ref ** 2).sum(axis=-1))
    rel = num / np.maximum(den, 1e-30)
    rel = np.where(den == 0, np.where(num == 0, 0.0, np.inf), rel)
    worst_rel = rel.max() if rel.size else 0.0
    assert worst_rel <= row_rel, f"{what}: per-row relative L2 error {worst_rel:.3e} > {row_rel}"
    return worst, worst_rel


def check_lse(gpu, ref, what: str, tol: float = LSE_ABS):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    inf_ref = np.isneginf(ref)
    assert np.array_equal(np.isneginf(gpu), inf_ref), f"{what}: -inf pattern differs"
    d = np.abs(gpu[~inf_ref] - ref[~inf_ref])
    worst = d.max() if d.size else 0.0
    assert worst <= tol, f"{what}: lse error {worst:.3e} > {tol}"
    return worst
