"""Multi-round driver (Algorithm 1 with a synthetic optimiser) against the same loop run with
the CPU oracle: synchronisation decisions, estimates and the communication account."""
import numpy as np
import pytest

import fda_synth as S
from fda_testlib import REL

pytestmark = pytest.mark.gpu


def oracle_rounds(oracle, w, w_t0, xi, coeffs, l, m, drifts, variant, eps, theta, refresh_xi):
    w, w_t0 = w.copy(), w_t0.copy()
    xi = None if xi is None else xi.copy()
    out = {"H": [], "syncs": [], "tol": []}
    for t, dr in enumerate(drifts):
        w += dr
        st = oracle.local_state(w, w_t0, xi if variant == 0 else None, coeffs, l if variant == 1 else 0,
                                m if variant == 1 else 0)
        full = np.zeros((w.shape[0], 2 + l * m))
        full[:, :st.shape[1]] = st
        est = oracle.combine(full, l, m, variant, eps, theta)
        out["H"].append(est["H"])
        out["tol"].append(4 * REL * (abs(est["mean_sq"]) + abs(est["est"])))
        if est["trigger"]:
            avg = oracle.average(w)
            if refresh_xi:
                xi = oracle.direction(avg, w_t0).astype(np.float32)
            w_t0 = avg.astype(np.float32)
            w[:] = w_t0
            out["syncs"].append(t)
    return out


@pytest.mark.parametrize("variant,theta,refresh,averaged", [
    (1, 2e-3, False, False), (1, 2e-3, False, True), (0, 2e-3, True, False), (0, 0.0, False, False),
    (1, 0.0, False, True), (0, 1e9, False, False),
])
def test_rounds_follow_the_oracle(variant, theta, refresh, averaged):
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    import oracle
    import paper_2405_20988_b200 as F

    rng = np.random.default_rng(77)
    K, d, l, m, steps, eps = 6, 20_011, 5, 250, 14, 0.06
    coeffs = S.hash_coefficients(5, l)
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    w_np = np.tile(w_t0, (K, 1))
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    common = rng.normal(0, 2e-4, size=(steps, 1, d)).astype(np.float32)       # a shared direction of progress
    drifts = (common + rng.normal(0, 2e-4, size=(steps, K, d))).astype(np.float32)
    ref = oracle_rounds(oracle, w_np, w_t0, xi, coeffs, l, m, drifts, variant, eps, float(np.float32(theta)), refresh)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w = torch.from_numpy(w_np.copy()).cuda()
        w0 = torch.from_numpy(w_t0.copy()).cuda()
        xg = torch.from_numpy(xi.copy()).cuda()
        dev = torch.from_numpy(drifts).cuda()
        got = F.run_rounds(ctx, w, w0, xg, steps, lambda t, ww: ww.add_(dev[t]), variant, eps, theta,
                           refresh_xi=refresh, averaged_state=averaged)
    # decisions agree unless an estimate sits within tolerance of Theta (then later steps may differ)
    for t in range(steps):
        assert abs(got["H"][t] - ref["H"][t]) <= ref["tol"][t] * (3 if averaged else 1) + 1e-12
        near = abs(ref["H"][t] - theta) <= ref["tol"][t] * 3
        if near:
            break
        assert (t in got["syncs"]) == (t in ref["syncs"])
    else:
        assert got["syncs"] == ref["syncs"]
        per_state = 4 * (1 + (l * m if variant == 1 else 1))
        assert got["state_bytes"] == steps * K * per_state
        assert got["model_bytes"] == len(ref["syncs"]) * K * d * 4
    if theta == 0.0:
        assert got["syncs"] == list(range(steps))        # Theta = 0 is the Synchronous scheme
    if theta == 1e9:
        assert got["syncs"] == []


@pytest.mark.parametrize("variant,refresh,averaged", [(1, False, False), (1, False, True), (0, True, False)])
def test_rounds_replayed_from_a_graph_give_the_eager_bits(variant, refresh, averaged):
    """graph=True records the library calls of a step once and replays them: the same estimates,
    synchronisation steps, account and final models, bit for bit, as the eager loop."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    import paper_2405_20988_b200 as F

    rng = np.random.default_rng(78)
    K, d, l, m, steps, eps, theta = 6, 20_011, 5, 250, 14, 0.06, 2e-3
    coeffs = S.hash_coefficients(6, l)
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    common = rng.normal(0, 2e-4, size=(steps, 1, d)).astype(np.float32)
    dev = torch.from_numpy((common + rng.normal(0, 2e-4, size=(steps, K, d))).astype(np.float32)).cuda()
    results = []
    for graph in (False, True):
        with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
            w = torch.from_numpy(np.tile(w_t0, (K, 1))).cuda()
            w0 = torch.from_numpy(w_t0.copy()).cuda()
            xg = torch.from_numpy(xi.copy()).cuda()
            got = F.run_rounds(ctx, w, w0, xg, steps, lambda t, ww: ww.add_(dev[t]), variant, eps, theta,
                               refresh_xi=refresh, averaged_state=averaged, graph=graph)
            torch.cuda.synchronize()
            results.append((got, w.cpu().numpy(), w0.cpu().numpy(), xg.cpu().numpy()))
    (a, wa, w0a, xa), (b, wb, w0b, xb) = results
    assert a["H"] == b["H"] and a["syncs"] == b["syncs"] and 0 < len(a["syncs"]) < steps
    assert a["state_bytes"] == b["state_bytes"] and a["model_bytes"] == b["model_bytes"]
    assert np.array_equal(wa, wb) and np.array_equal(w0a, w0b) and np.array_equal(xa, xb)
