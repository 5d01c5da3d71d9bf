"""Pins for the CPU oracle: every check here compares it with something that is not the
oracle itself - arbitrary-precision integer arithmetic, closed forms, numpy brute force,
identities and guarantees stated in the paper (Section 3, Eq. 2-4, Theorems 1 and 2)."""
import os

import numpy as np
import pytest

import fda_synth as S
import oracle

P = (1 << 61) - 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def py_bucket(c, j, m):
    return ((int(c[0]) * j + int(c[1])) % P) % m


def py_sign(c, j):
    g = (int(c[2]) * j + int(c[3])) % P
    g = (g * j + int(c[4])) % P
    g = (g * j + int(c[5])) % P
    return -1 if g & 1 else 1


def rand_coeffs(rng, l):
    c = rng.integers(0, P, size=6 * l, dtype=np.uint64)
    c[0::6] |= np.uint64(1)
    c[2::6] |= np.uint64(1)
    return c


def injective_coeffs(l):
    """a=1, b=0: bucket(j) = j for j < m (closed form); arbitrary sign polynomial."""
    c = np.zeros(6 * l, dtype=np.uint64)
    for i in range(l):
        c[6 * i:6 * i + 6] = [1, 0, 3 + i, 5 + 2 * i, 7 + i, 11 + i]
    return c


def states_of(w, w_t0, xi, c, l, m):
    return oracle.local_state(np.ascontiguousarray(w, dtype=np.float32), w_t0, xi, c, l, m)


# ------------------------------------------------------------------------------- hash
def test_hash_matches_big_integer_arithmetic():
    rng = np.random.default_rng(7)
    l, m = 6, 250
    c = rand_coeffs(rng, l)
    js = [0, 1, 2, 249, 250, 61_705, 197_767_335, (1 << 31) - 1, (1 << 31), (1 << 40) + 12345]
    js += [int(x) for x in rng.integers(0, 1 << 28, size=200)]
    for j in js:
        b, s = oracle.hash_dump(c, l, m, j, 3)
        for i in range(l):
            for t in range(3):
                assert b[i, t] == py_bucket(c[6 * i:6 * i + 6], j + t, m)
                assert s[i, t] == py_sign(c[6 * i:6 * i + 6], j + t)


def test_hash_edge_coefficients_and_residues():
    m = 250
    j = 123_456_789
    # extreme coefficients
    for a in (1, P - 1, P - 2, 1 << 60):
        for b in (0, P - 1):
            c = np.array([a, b, P - 1, P - 1, P - 1, P - 1], dtype=np.uint64)
            bk, sg = oracle.hash_dump(c, 1, m, j, 2)
            assert bk[0, 0] == py_bucket(c, j, m) and sg[0, 0] == py_sign(c, j)
            assert bk[0, 1] == py_bucket(c, j + 1, m) and sg[0, 1] == py_sign(c, j + 1)
    # residues 0 and p-1 of the bucket polynomial: choose b so that a*j+b = 0 or p-1 (mod p)
    a = 0x0123456789ABCDE % P
    for target in (0, P - 1, 1, m - 1, m):
        b = (target - a * j) % P
        c = np.array([a, b, 1, 0, 0, 0], dtype=np.uint64)
        bk, _ = oracle.hash_dump(c, 1, m, j, 1)
        assert bk[0, 0] == target % m
    # residues 0, 1, p-1, p-2 of the sign polynomial: choose c0
    c3, c2, c1 = 0x1555555555555555 % P, 12345, 67890
    base = (((c3 * j + c2) % P) * j + c1) % P * j % P
    for target, sign in ((0, 1), (1, -1), (P - 1, 1), (P - 2, -1)):
        c0 = (target - base) % P
        c = np.array([1, 0, c3, c2, c1, c0], dtype=np.uint64)
        _, sg = oracle.hash_dump(c, 1, m, j, 1)
        assert sg[0, 0] == sign


def test_hash_closed_forms():
    m, n = 37, 500
    # a=1, b=0 -> bucket = j mod m;  g = j^3 (c3=1, rest 0) -> parity of j for j^3 < p
    c = np.array([1, 0, 1, 0, 0, 0], dtype=np.uint64)
    bk, sg = oracle.hash_dump(c, 1, m, 0, n)
    j = np.arange(n)
    assert np.array_equal(bk[0], j % m)
    assert np.array_equal(sg[0], np.where(j % 2 == 0, 1, -1))
    # a = p-1 = -1: y = (b - j) mod p with b = 1000 -> 1000-j for j<=1000
    c = np.array([P - 1, 1000, 1, 0, 0, 1], dtype=np.uint64)
    bk, sg = oracle.hash_dump(c, 1, m, 0, n)
    assert np.array_equal(bk[0], (1000 - j) % m)
    assert np.array_equal(sg[0], np.where((j + 1) % 2 == 0, 1, -1))   # j^3 + 1


def test_bucket_and_sign_balance():
    """2-wise bucket hash spreads indices evenly and signs are balanced (loose chi-square)."""
    rng = np.random.default_rng(3)
    l, m, n = 4, 250, 200_000
    c = rand_coeffs(rng, l)
    bk, sg = oracle.hash_dump(c, l, m, 0, n)
    for i in range(l):
        cnt = np.bincount(bk[i], minlength=m)
        chi2 = np.sum((cnt - n / m) ** 2 / (n / m))
        assert chi2 < m + 6 * np.sqrt(2 * m)
        assert abs(int(sg[i].sum())) < 6 * np.sqrt(n)


# ----------------------------------------------------------------------- golden (paper)
def test_recommended_sketch_size_is_5kB():
    rows = [r.split() for r in open(os.path.join(GOLDEN, "sketch_size.txt")) if not r.startswith("#")]
    l, m, cell, total = map(int, rows[0])
    assert (oracle.state_len(l, m) - 2) * cell == total == 5000


# ----------------------------------------------------------------------------- sketch
def test_sketch_of_basis_vectors_reads_back_bucket_and_sign():
    rng = np.random.default_rng(11)
    d, l, m = 300, 5, 31
    c = rand_coeffs(rng, l)
    w_t0 = np.zeros(d, dtype=np.float32)
    for j in (0, 1, 17, 299):
        w = np.zeros((1, d), dtype=np.float32)
        w[0, j] = 2.5
        st = states_of(w, w_t0, None, c, l, m)[0]
        assert st[0] == 6.25 and st[1] == 0.0
        sk = st[2:].reshape(l, m)
        for i in range(l):
            nz = np.flatnonzero(sk[i])
            assert list(nz) == [py_bucket(c[6 * i:6 * i + 6], j, m)]
            assert sk[i, nz[0]] == 2.5 * py_sign(c[6 * i:6 * i + 6], j)


def test_sketch_linearity_exact_on_integers():
    rng = np.random.default_rng(5)
    d, l, m = 4000, 5, 64
    c = rand_coeffs(rng, l)
    a = rng.integers(-50, 51, size=d).astype(np.float32)
    b = rng.integers(-50, 51, size=d).astype(np.float32)
    z = np.zeros(d, dtype=np.float32)
    sa = states_of(a[None], z, None, c, l, m)[0, 2:]
    sb = states_of(b[None], z, None, c, l, m)[0, 2:]
    sab = states_of((3 * a - 2 * b)[None], z, None, c, l, m)[0, 2:]
    assert np.array_equal(3 * sa - 2 * sb, sab)
    # the drift, not the model, is sketched: shifting w and w_t0 together changes nothing
    shift = rng.integers(-8, 9, size=d).astype(np.float32)
    assert np.array_equal(states_of((a + shift)[None], shift, None, c, l, m)[0, 2:], sa)


def test_sketch_zero_and_signed_column_sums():
    rng = np.random.default_rng(6)
    d, l, m = 1500, 3, 50
    c = rand_coeffs(rng, l)
    z = np.zeros(d, dtype=np.float32)
    assert not states_of(z[None], z, None, c, l, m).any()
    v = rng.integers(-9, 10, size=d).astype(np.float32)
    sk = states_of(v[None], z, None, c, l, m)[0, 2:].reshape(l, m)
    for i in range(l):
        signed = sum(py_sign(c[6 * i:6 * i + 6], j) * float(v[j]) for j in range(d))
        assert sk[i].sum() == signed


def test_injective_buckets_recover_the_norm_and_the_variance_exactly():
    rng = np.random.default_rng(8)
    K, d, l, m = 4, 40, 5, 64          # d <= m and bucket(j) = j: no collisions
    c = injective_coeffs(l)
    w_t0 = rng.integers(-5, 6, size=d).astype(np.float32)
    w = (w_t0 + rng.integers(-7, 8, size=(K, d))).astype(np.float32)
    st = states_of(w, w_t0, None, c, l, m)
    u = w.astype(np.float64) - w_t0
    for k in range(K):
        rows = (st[k, 2:].reshape(l, m) ** 2).sum(1)
        assert np.all(rows == (u[k] ** 2).sum()) and st[k, 0] == (u[k] ** 2).sum()
    est = oracle.combine(st, l, m, 1, 0.0, 0.0)
    var = np.mean(((u - u.mean(0)) ** 2).sum(1))
    assert est["H"] == pytest.approx(var, rel=1e-13)
    assert est["est"] == pytest.approx((u.mean(0) ** 2).sum(), rel=1e-13)


def test_ams_estimator_moments():
    """Each row norm is an unbiased estimate of ||v||^2 with variance 2(||v||_2^4-||v||_4^4)/m
    (the F2 estimator behind M2 in Section 3.1), checked over many coefficient tables."""
    rng = np.random.default_rng(2024)
    d, m, l, tables = 120, 16, 8, 400
    v = rng.normal(size=d).astype(np.float32)
    z = np.zeros(d, dtype=np.float32)
    n2 = float(np.sum(v.astype(np.float64) ** 2))
    n4 = float(np.sum(v.astype(np.float64) ** 4))
    rows = []
    for _ in range(tables):
        c = rand_coeffs(rng, l)
        sk = states_of(v[None], z, None, c, l, m)[0, 2:].reshape(l, m)
        rows.extend((sk ** 2).sum(1))
    rows = np.array(rows)
    var_theory = 2.0 * (n2 * n2 - n4) / m
    se = np.sqrt(var_theory / rows.size)
    assert abs(rows.mean() - n2) < 4.5 * se
    assert rows.var() == pytest.approx(var_theory, rel=0.15)


# ------------------------------------------------------------- norms, projection, Eq. 4
def test_variance_identity_by_brute_force():
    rng = np.random.default_rng(9)
    K, d = 7, 1003
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    w = (w_t0 + rng.normal(0, 1e-3, size=(K, d))).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    st = states_of(w, w_t0, xi, None, 0, 0)
    W, W0 = w.astype(np.float64), w_t0.astype(np.float64)
    u = W - W0
    var_def = np.mean(((W - W.mean(0)) ** 2).sum(1))                       # Eq. (2)
    assert st[:, 0] == pytest.approx((u ** 2).sum(1), rel=1e-12)
    assert st[:, 1] == pytest.approx(u @ xi.astype(np.float64), rel=1e-9, abs=1e-15)
    assert st[:, 0].mean() - (u.mean(0) ** 2).sum() == pytest.approx(var_def, rel=1e-9)   # Eq. (4)
    v = oracle.variance(w, w_t0)
    assert v[0] == pytest.approx(var_def, rel=1e-12)
    assert v[1] - v[2] == pytest.approx(var_def, rel=1e-9)


def test_linear_bound_holds_and_is_tight_for_parallel_xi():
    rng = np.random.default_rng(10)
    K, d = 6, 700
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    w = (w_t0 + rng.normal(2e-4, 1e-3, size=(K, d))).astype(np.float32)
    u = w.astype(np.float64) - w_t0
    var = np.mean(((u - u.mean(0)) ** 2).sum(1))
    for trial in range(20):
        xi = rng.normal(size=d)
        xi = (xi / np.linalg.norm(xi)).astype(np.float32)
        H = oracle.combine(states_of(w, w_t0, xi, None, 0, 0), 0, 0, 0, 0.0, 0.0)["H"]
        assert H >= var * (1 - 1e-6)            # Theorem 2 (xi is unit only to fp32 rounding)
    xi = u.mean(0) / np.linalg.norm(u.mean(0))   # equality case of Cauchy-Schwarz
    est = oracle.combine(states_of(w, w_t0, xi.astype(np.float32), None, 0, 0), 0, 0, 0, 0.0, 0.0)
    assert est["H"] == pytest.approx(var, rel=1e-5)
    assert est["est"] == pytest.approx((u.mean(0) ** 2).sum(), rel=1e-6)


def test_sketch_bound_holds_with_high_probability():
    """Theorem 1: H >= Var with probability >= 1-delta.  With 5 x 250 and eps = 0.06 the
    F2 moments predict about 0.9 for the one-sided event; the paper quotes ~95 % two-sided
    confidence empirically.  The observed rate must clear 0.8."""
    rng = np.random.default_rng(12)
    K, d, l, m, eps, trials = 5, 3000, 5, 250, 0.06, 120
    ok = 0
    for _ in range(trials):
        c = rand_coeffs(rng, l)
        w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
        w = (w_t0 + rng.normal(3e-4, 1e-3, size=(K, d))).astype(np.float32)
        u = w.astype(np.float64) - w_t0
        var = np.mean(((u - u.mean(0)) ** 2).sum(1))
        ok += oracle.combine(states_of(w, w_t0, None, c, l, m), l, m, 1, eps, 0.0)["H"] >= var
    assert ok / trials >= 0.8


# ----------------------------------------------------------------- combine and trigger
def test_combine_median_and_strict_trigger():
    l, m, K = 4, 3, 2
    st = np.zeros((K, 2 + l * m))
    st[:, 0] = [10.0, 14.0]                     # mean 12
    st[:, 1] = [1.0, 3.0]                       # mean 2 -> linear est 4
    rows = [[1, 0, 0], [0, 2, 0], [0, 0, 3], [2, 2, 1]]      # row norms^2 1, 4, 9, 9
    for k in range(K):
        st[k, 2:] = np.array(rows, dtype=float).reshape(-1)
    sk = oracle.combine(st, l, m, 1, 0.25, 6.8)
    assert list(sk["rows"]) == [1.0, 4.0, 9.0, 9.0]
    assert sk["est"] == pytest.approx(6.5 / 1.25)            # even l: mean of 4 and 9
    assert sk["H"] == pytest.approx(12 - 5.2) and sk["mean_sq"] == 12.0
    lin = oracle.combine(st, l, m, 0, 0.25, 8.0)
    assert lin["H"] == 8.0 and lin["trigger"] is False       # strict '>' (Algorithm 1)
    assert oracle.combine(st, l, m, 0, 0.25, np.nextafter(8.0, 0))["trigger"] is True
    odd = oracle.combine(st[:, :2 + 3 * m], 3, m, 1, 0.0, 0.0)
    assert odd["est"] == 4.0                                 # odd l: the middle value
    # Theta = 0 is the Synchronous special case: fires as soon as H > 0
    assert oracle.combine(st, l, m, 0, 0.0, 0.0)["trigger"] is True


def test_state_after_synchronisation_is_zero():
    rng = np.random.default_rng(13)
    K, d, l, m = 4, 900, 5, 40
    c = rand_coeffs(rng, l)
    w = rng.integers(-64, 65, size=(K, d)).astype(np.float32)     # K = 4: mean exact in fp32
    wbar = oracle.average(w)
    assert np.array_equal(wbar, w.astype(np.float64).mean(0))
    synced = np.tile(wbar.astype(np.float32), (K, 1))
    st = states_of(synced, wbar.astype(np.float32), np.ones(d, np.float32), c, l, m)
    assert not st.any()
    est = oracle.combine(st, l, m, 1, 0.06, 0.0)
    assert est["H"] == 0.0 and est["trigger"] is False


def test_average_special_cases():
    rng = np.random.default_rng(14)
    w = rng.normal(size=(1, 77)).astype(np.float32)
    assert np.array_equal(oracle.average(w), w[0].astype(np.float64))       # K = 1
    w = rng.normal(size=(5, 64)).astype(np.float32)
    buf = np.zeros((5, 96), dtype=np.float32)
    buf[:, :64] = w
    assert np.allclose(oracle.average(buf[:, :64]), w.astype(np.float64).mean(0), rtol=1e-15)
    assert np.array_equal(oracle.average(buf[:, :64], 10, 20), oracle.average(buf[:, :64])[10:20])


# ------------------------------------------------------- workload-level closed forms
@pytest.mark.parametrize("idx, mean_sq, ubar_sq", [(1, 0.061706, 0.0123412), (2, 1.4998525, 0.4199587)])
def test_workload_expectations(idx, mean_sq, ubar_sq):
    """Closed forms of the input recipe: E||u_k||^2 = d*sigma^2 (+ d*5e-4^2 shared) and
    E||u-bar||^2 = d*sigma^2/K (+ d*5e-4^2)."""
    wl = S.WORKLOADS[idx]
    w_t0 = S.last_global_model(wl)
    w = S.worker_models(wl, w_t0)[:, :wl.d]
    xi = S.unit_direction(wl)
    c = S.hash_coefficients(wl.seed, wl.l)
    st = oracle.local_state(w, w_t0, xi, c, wl.l, wl.m, threads=4)
    var, msq, ub = oracle.variance(w, w_t0)
    tol = 6.0 / np.sqrt(wl.d)
    assert st[:, 0].mean() == pytest.approx(mean_sq, rel=tol + 1e-3)
    assert msq == pytest.approx(st[:, 0].mean(), rel=1e-9)
    assert ub == pytest.approx(ubar_sq, rel=tol * np.sqrt(2) + 2e-3)
    sk = oracle.combine(st, wl.l, wl.m, 1, wl.epsilon, wl.thetas[-1])
    lin = oracle.combine(st, wl.l, wl.m, 0, wl.epsilon, wl.thetas[-1])
    assert lin["H"] >= var * (1 - 1e-6)
    assert sk["est"] * (1 + wl.epsilon) == pytest.approx(ub, rel=0.25)
    assert sk["trigger"] and lin["trigger"]


def test_direction_heuristic_closed_forms():
    """xi = (w_new - w_old)/||.|| (Section 3.2): a 3-4-5 step, unit norm, parallelism, zero step."""
    old = np.array([1.0, 2.0, 3.0, 4.0], dtype=np.float32)
    new = old.astype(np.float64) + np.array([3.0, 0.0, -4.0, 0.0])
    assert np.allclose(oracle.direction(new, old), [0.6, 0.0, -0.8, 0.0], rtol=0, atol=1e-15)
    rng = np.random.default_rng(15)
    old = rng.normal(size=1000).astype(np.float32)
    new = old.astype(np.float64) + rng.normal(0, 1e-3, size=1000)
    xi = oracle.direction(new, old)
    step = new - old
    assert np.sum(xi * xi) == pytest.approx(1.0, rel=1e-13)
    assert xi @ step == pytest.approx(np.linalg.norm(step), rel=1e-13)      # parallel, same sense
    assert not oracle.direction(old.astype(np.float64), old).any()
