"""Shared test helpers: the near-threshold band rule for index sets and error measures."""
import numpy as np


def check_topk_band(gpu_idx, oracle_idx, scores, cand, rel_band, scale_ref=None, what=""):
    """Index-set parity with the near-threshold exclusion.

    scores: oracle scores (float64) indexable by position; cand: candidate positions.  The k-th largest
    oracle score is the threshold tau; positions whose score lies within delta = rel_band * |scale_ref or
    tau| of tau may legitimately differ (the GPU ranks float32 scores).  Everything else must agree
    exactly.  Returns the number of candidates inside the band."""
    gpu = [int(i) for i in gpu_idx if i >= 0]
    ora = [int(i) for i in oracle_idx]
    assert gpu == sorted(gpu) and len(set(gpu)) == len(gpu), f"{what}: not ascending/unique"
    assert len(gpu) == len(ora), f"{what}: size {len(gpu)} != {len(ora)}"
    if not ora:
        return 0
    cand = list(cand)
    assert set(gpu) <= set(cand), f"{what}: pick outside the candidate range"
    tau = min(float(scores[i]) for i in ora)
    delta = rel_band * abs(tau if scale_ref is None else scale_ref)
    for i in gpu:
        assert float(scores[i]) >= tau - delta, f"{what}: pick {i} scores below the band"
    must = {i for i in cand if float(scores[i]) > tau + delta}
    assert must <= set(gpu), f"{what}: clear winners missing: {sorted(must - set(gpu))[:8]}"
    band = {i for i in cand if abs(float(scores[i]) - tau) <= delta}
    assert set(gpu) - band == set(ora) - band, f"{what}: sets differ outside the band"
    return len(band)


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)))) if np.size(a) else 0.0


def rel_rms(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = float(np.sqrt(np.mean(b * b)))
    return float(np.sqrt(np.mean((a - b) ** 2))) / den if den > 0 else 0.0
