"""Shared helpers for the GPU parity tests: tolerances and oracle/GPU comparison."""
import numpy as np

REL = 1e-5   # relative tolerance on norms, projections, sketch cells and averaged weights


def check_states(gpu_states, ora_states, l, m, d, xi_norm=1.0, rows=None, flags_sketch=True):
    """Element-by-element comparison of local states (fp32 GPU vs fp64 oracle).

    norm        |err| <= REL * oracle
    projection  |err| <= REL * max(|oracle|, sqrt(n_k/d) * ||xi||)   (scale of a random projection)
    sketch cell |err| <= REL * max(|oracle cell|, sqrt(n_k/m))        (rms size of a cell)
    """
    g = np.asarray(gpu_states, dtype=np.float64)
    o = np.asarray(ora_states, dtype=np.float64)
    ks = range(o.shape[0]) if rows is None else rows
    worst = {"norm": 0.0, "proj": 0.0, "cell": 0.0}
    for k in ks:
        n = o[k, 0]
        worst["norm"] = max(worst["norm"], abs(g[k, 0] - n) / max(n, 1e-300))
        pscale = max(abs(o[k, 1]), np.sqrt(n / d) * xi_norm, 1e-300)
        worst["proj"] = max(worst["proj"], abs(g[k, 1] - o[k, 1]) / pscale)
        if l > 0 and flags_sketch:
            scale = np.maximum(np.abs(o[k, 2:]), np.sqrt(n / m))
            scale = np.maximum(scale, 1e-300)
            worst["cell"] = max(worst["cell"], float(np.max(np.abs(g[k, 2:] - o[k, 2:]) / scale)))
    assert worst["norm"] <= REL, worst
    assert worst["proj"] <= REL, worst
    assert worst["cell"] <= REL, worst
    return worst


def check_estimate(gpu_est, ora_est, l):
    """H = A - B is compared with |err| <= REL * (|A| + |B|) (each term carries REL)."""
    assert abs(gpu_est["mean_sq"] - ora_est["mean_sq"]) <= REL * abs(ora_est["mean_sq"]) + 1e-37
    assert abs(gpu_est["est"] - ora_est["est"]) <= REL * abs(ora_est["est"]) + 1e-37
    tol_h = REL * (abs(ora_est["mean_sq"]) + abs(ora_est["est"])) + 1e-37
    assert abs(gpu_est["H"] - ora_est["H"]) <= tol_h
    if l > 0:
        assert np.allclose(gpu_est["rows"], ora_est["rows"], rtol=REL, atol=1e-37)
    return tol_h


def check_trigger(gpu_est, ora_est, theta, tol_h):
    """Decisions must agree unless the estimate lies within tolerance of Theta."""
    if abs(ora_est["H"] - theta) > tol_h + REL * abs(theta):
        assert gpu_est["trigger"] == ora_est["trigger"]


def check_average(gpu_avg, ora_avg, mean_abs=None):
    g = np.asarray(gpu_avg, dtype=np.float64)
    o = np.asarray(ora_avg, dtype=np.float64)
    scale = np.maximum(np.abs(o), np.mean(np.abs(o)) if mean_abs is None else mean_abs)
    scale = np.maximum(scale, 1e-300)
    err = float(np.max(np.abs(g - o) / scale)) if o.size else 0.0
    assert err <= REL, err
    return err


def check_mean_state(gpu_mean, ora_states, ubar_sq, l, m, d, K, sketch=True):
    """Averaged state S-bar (fp32, one pass on the GPU) against the mean of the oracle's K
    states, at the same relative tolerance as the per-worker states.  Scales: the averaged
    projection and the cells of sk(u-bar) have the size of a random projection / sketch cell of
    u-bar, so they are compared relative to max(|value|, sqrt(||u-bar||^2/d)) and
    max(|cell|, sqrt(||u-bar||^2/m)).  (Measured on B200 over the seven synthetic workloads: the
    worst cell is off by 1.4e-6 of that scale, the worst projection by 1.0e-7.)  Returns the
    worst ratios."""
    g = np.asarray(gpu_mean, dtype=np.float64)
    o = np.asarray(ora_states, dtype=np.float64).mean(axis=0)
    worst = {"norm": abs(g[0] - o[0]) / max(o[0], 1e-300)}
    assert abs(g[0] - o[0]) <= REL * o[0] + 1e-300
    pscale = max(abs(o[1]), np.sqrt(ubar_sq / d), 1e-300)
    worst["proj"] = abs(g[1] - o[1]) / pscale
    assert worst["proj"] <= REL, worst
    if l > 0 and sketch:
        scale = np.maximum(np.maximum(np.abs(o[2:]), np.sqrt(ubar_sq / m)), 1e-300)
        worst["cell"] = float(np.max(np.abs(g[2:] - o[2:]) / scale))
        assert worst["cell"] <= REL, worst
    return worst


def mean_estimate_tolerance(ref, ubar_sq):
    """Tolerance on H of the averaged state: REL on the mean squared norm, and on the estimate of
    ||u-bar||^2 the bound that follows from cells within REL of max(|cell|, rms cell):
    |sum of squares - reference| <= 2 REL (sum cell^2 + m rms^2) <= 4 REL max(estimate, ||u-bar||^2)."""
    return REL * abs(ref["mean_sq"]) + 4 * REL * max(abs(ref["est"]), ubar_sq) + 1e-37
