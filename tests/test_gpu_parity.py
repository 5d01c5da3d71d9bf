"""GPU parity: libfda (through its C ABI) against the CPU oracle, element by element."""
import os

import numpy as np
import pytest

import fda_synth as S
from fda_testlib import (REL, check_average, check_estimate, check_mean_state, check_states, check_trigger,
                         mean_estimate_tolerance)

HOST_CORES = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)

pytestmark = pytest.mark.gpu

P = (1 << 61) - 1


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    import oracle
    import paper_2405_20988_b200 as F
    F.load_library()
    return torch, oracle, F


def rand_coeffs(rng, l):
    c = rng.integers(0, P, size=6 * l, dtype=np.uint64)
    c[0::6] |= np.uint64(1)
    c[2::6] |= np.uint64(1)
    return c


ALL = 1 | 2 | 4


def gpu_states(torch, F, ctx, w_np, w_t0_np, xi_np, flags=ALL, misalign=0):
    """Run fda_local_state on host arrays (optionally at a misaligned device offset)."""
    K, stride = w_np.shape[0], w_np.shape[1]

    def put(a):
        if a is None:
            return None
        buf = torch.empty(a.size + 8, dtype=torch.float32, device="cuda")
        view = buf[misalign:misalign + a.size].view(a.shape)
        view.copy_(torch.from_numpy(np.ascontiguousarray(a)))
        return view

    w, w0, xi = put(w_np), put(w_t0_np), put(xi_np)
    states = torch.full((K, ctx.state_len), float("nan"), dtype=torch.float32, device="cuda")
    return w, w0, xi, states


def run_case(env, K, d, l, m, seed, flags=ALL, misalign=0, stride=None, with_xi=True, sigma=1e-3):
    torch, oracle, F = env
    rng = np.random.default_rng(seed)
    stride = S.row_stride(d) if stride is None else stride
    coeffs = rand_coeffs(rng, l) if l > 0 else None
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    wbuf = np.zeros((K, stride), dtype=np.float32)
    wbuf[:, :d] = w_t0 + rng.normal(0, sigma, size=(K, d)).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32) if with_xi else None
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w, w0, xg, st = gpu_states(torch, F, ctx, wbuf, w_t0, xi, flags, misalign)
        ctx.fda_local_state(w[:, :d], w0, xg, flags, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi if (flags & 2) else None, coeffs,
                             l if (flags & 4) else 0, m if (flags & 4) else 0)
    full = np.zeros((K, 2 + l * m))
    full[:, :ora.shape[1]] = ora
    if not flags & 1:
        full[:, 0] = 0.0
        assert not got[:, 0].any()
        got = got.copy()
        got[:, 0] = 0
        n_for_scale = oracle.local_state(wbuf[:, :d], w_t0, None, None, 0, 0)[:, 0]
    if not flags & 4 and l > 0:
        assert not got[:, 2:].any()
    if flags & 1:
        check_states(got, full, l if flags & 4 else 0, m, d)
    else:                      # norm slot off: compare the rest against scales from the oracle norm
        full2 = full.copy(); full2[:, 0] = n_for_scale
        got2 = got.copy(); got2[:, 0] = n_for_scale
        check_states(got2, full2, l if flags & 4 else 0, m, d)
    return got, full


# ------------------------------------------------------------------------------- hash
def test_hash_dump_bit_exact(env):
    torch, oracle, F = env
    rng = np.random.default_rng(1)
    for l, m in ((5, 250), (7, 500), (16, 3000), (1, 32768), (1, 1), (3, 37)):
        coeffs = rand_coeffs(rng, l)
        if l >= 3:                          # extreme coefficient values in some rows
            coeffs[0:6] = [P - 1, P - 1, P - 1, P - 1, P - 1, P - 1]
            coeffs[6:12] = [1, 0, 1, 0, 0, 0]
        with F.FdaContext(l, m, coeffs, d_max=1024, K_max=1) as ctx:
            for j0, n in ((0, 5000), (61_700, 1000), (197_767_000, 4096), ((1 << 31) - 3000, 3000),
                          (int(rng.integers(0, 1 << 30)), 2048)):
                b = torch.empty((l, n), dtype=torch.int16, device="cuda")
                s = torch.empty((l, n), dtype=torch.int8, device="cuda")
                ctx.fda_debug_hash(j0, n, b, s)
                torch.cuda.synchronize()
                ob, os_ = oracle.hash_dump(coeffs, l, m, j0, n)
                assert np.array_equal(b.cpu().numpy().view(np.uint16).astype(np.int32), ob)
                assert np.array_equal(s.cpu().numpy(), os_)


def test_hash_residue_edges(env):
    """Coefficients chosen so that the bucket residue is 0 / p-1 and the sign residue is
    0, 1, p-1, p-2 at a given index: the canonical-form corner cases."""
    torch, oracle, F = env
    j, m = 123_456_789, 250
    a, c3, c2, c1 = 0x0123456789ABCDE % P, 0x1555555555555555 % P, 12345, 67890
    base = (((c3 * j + c2) % P) * j + c1) % P * j % P
    for tb in (0, P - 1, m, m - 1):
        for ts in (0, 1, P - 1, P - 2):
            coeffs = np.array([a, (tb - a * j) % P, c3, c2, c1, (ts - base) % P], dtype=np.uint64)
            with F.FdaContext(1, m, coeffs, d_max=64, K_max=1) as ctx:
                b = torch.empty((1, 4), dtype=torch.int16, device="cuda")
                s = torch.empty((1, 4), dtype=torch.int8, device="cuda")
                ctx.fda_debug_hash(j - 1, 4, b, s)
                torch.cuda.synchronize()
            ob, os_ = oracle.hash_dump(coeffs, 1, m, j - 1, 4)
            assert np.array_equal(b.cpu().numpy().view(np.uint16).astype(np.int32), ob)
            assert np.array_equal(s.cpu().numpy(), os_)
            assert ob[0, 1] == tb % m and os_[0, 1] == (-1 if ts & 1 else 1)


def test_sketch_of_basis_vectors_reads_back_the_table(env):
    """sk(alpha*e_j) has one non-zero per row at bucket_i(j) with value sign_i(j)*alpha: reads
    the hash the kernel really uses (its table) back out and compares it bit for bit."""
    torch, oracle, F = env
    rng = np.random.default_rng(2)
    d, l, m = 70_001, 5, 250
    coeffs = rand_coeffs(rng, l)
    js = [0, 1, 2, 3, 4, 63, 64, 1023, 1024, 8191, 8192, 70_000] + [int(x) for x in rng.integers(0, d, 20)]
    K = len(js)
    wbuf = np.zeros((K, S.row_stride(d)), dtype=np.float32)
    for r, j in enumerate(js):
        wbuf[r, j] = 1.5
    w_t0 = np.zeros(d, dtype=np.float32)
    ob, os_ = oracle.hash_dump(coeffs, l, m, 0, d)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w, w0, _, st = gpu_states(torch, F, ctx, wbuf, w_t0, None)
        ctx.fda_local_state(w[:, :d], w0, None, 1 | 4, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
    for r, j in enumerate(js):
        assert got[r, 0] == 2.25 and got[r, 1] == 0
        sk = got[r, 2:].reshape(l, m)
        for i in range(l):
            nz = np.flatnonzero(sk[i])
            assert list(nz) == [ob[i, j]]
            assert sk[i, nz[0]] == 1.5 * os_[i, j]


# ---------------------------------------------------------------------- small shapes
@pytest.mark.parametrize("K,d,l,m", [
    (1, 1, 5, 250), (1, 3, 5, 250), (2, 5, 3, 7), (5, 1000, 5, 250), (5, 4099, 5, 250),
    (8, 33_001, 5, 250), (10, 20_003, 5, 250), (30, 9_999, 5, 250), (33, 7_001, 5, 250),
    (60, 12_345, 7, 500), (17, 5_000, 7, 500), (3, 2_000, 16, 1000), (4, 3_000, 2, 20_000),
    (9, 2_500, 1, 1), (64, 1_111, 4, 64),
])
def test_local_state_small_shapes(env, K, d, l, m):
    run_case(env, K, d, l, m, seed=K * 1000 + d)


@pytest.mark.parametrize("misalign,stride_extra", [(1, 0), (3, 1), (0, 2), (2, 3)])
def test_local_state_unaligned_inputs(env, misalign, stride_extra):
    d = 10_007
    run_case(env, 6, d, 5, 250, seed=77 + misalign, misalign=misalign, stride=d + stride_extra)


@pytest.mark.parametrize("flags", [1, 2, 4, 1 | 2, 1 | 4, 2 | 4])
def test_local_state_flag_subsets(env, flags):
    run_case(env, 7, 6_001, 5, 250, seed=5, flags=flags)


def test_local_state_without_xi_and_without_sketch_context(env):
    got, _ = run_case(env, 4, 3_333, 5, 250, seed=6, with_xi=False)
    assert not got[:, 1].any()
    got, _ = run_case(env, 4, 3_333, 0, 0, seed=7, flags=1 | 2)
    assert got.shape[1] == 2


def test_heavy_tailed_values(env):
    """Outliers four orders of magnitude above the bulk (the heavy-tailed workload's shape)."""
    torch, oracle, F = env
    wl = S.small_workload(seed=3, d=200_003, K=12, l=7, m=500, drift="heavy")
    w_t0 = S.last_global_model(wl)
    wbuf = S.worker_models(wl, w_t0)
    xi = S.unit_direction(wl)
    coeffs = S.hash_coefficients(wl.seed, wl.l)
    with F.FdaContext(wl.l, wl.m, coeffs, d_max=wl.d, K_max=wl.K) as ctx:
        w, w0, xg, st = gpu_states(torch, F, ctx, wbuf, w_t0, xi)
        ctx.fda_local_state(w[:, :wl.d], w0, xg, ALL, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
    ora = oracle.local_state(wbuf[:, :wl.d], w_t0, xi, coeffs, wl.l, wl.m, threads=4)
    check_states(got, ora, wl.l, wl.m, wl.d)


# ------------------------------------------------------------------- averaged state
@pytest.mark.parametrize("K,d,l,m,misalign", [
    (1, 1, 5, 250, 0), (2, 7, 3, 7, 0), (5, 4099, 5, 250, 0), (8, 100_003, 5, 250, 0), (30, 20_001, 5, 250, 0),
    (60, 30_011, 7, 500, 0), (9, 9_999, 16, 1000, 0), (13, 10_007, 5, 250, 3), (4, 3_000, 2, 20_000, 0),
    (6, 40_000, 3, 100, 0), (18, 100_001, 7, 500, 1), (20, 100, 7, 500, 0), (3, 5, 7, 500, 1), (2, 5121, 7, 500, 0),
    # long vectors with few workers: the one-pass route on the list kernel (it needs eight tiles per SM)
    (3, 7_400_003, 5, 250, 0), (5, 7_300_001, 5, 250, 1), (10, 7_280_000, 5, 250, 0),
])
def test_mean_state_matches_mean_of_oracle_states(env, K, d, l, m, misalign):
    """sk(u-bar) = mean_k sk(u_k) (linearity, Section 3.1): the one-pass averaged state against
    the average of the oracle's per-worker states, and the estimate it leads to."""
    torch, oracle, F = env
    rng = np.random.default_rng(K * 7919 + d)
    stride = S.row_stride(d) + (1 if misalign else 0)
    coeffs = rand_coeffs(rng, l)
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    wbuf = np.zeros((K, stride), dtype=np.float32)
    wbuf[:, :d] = w_t0 + (rng.normal(2e-4, 1e-3, size=(K, d))).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, l, m, threads=4)
    _, _, ubar_sq = oracle.variance(wbuf[:, :d], w_t0)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w, w0, xg, _ = gpu_states(torch, F, ctx, wbuf, w_t0, xi, ALL, misalign)
        mean = torch.full((ctx.state_len,), float("nan"), dtype=torch.float32, device="cuda")
        buf = ctx.new_estimate_buffer()
        for flags in (ALL, 1 | 4, 1 | 2):
            ctx.fda_mean_state(w[:, :d], w0, xg, flags, mean)
            torch.cuda.synchronize()
            got = mean.cpu().numpy()
            ref = ora.copy()
            if not flags & 2:
                ref[:, 1] = 0
            if not flags & 4:
                assert not got[2:].any()
            check_mean_state(got, ref, ubar_sq, l, m, d, K, sketch=bool(flags & 4))
        ctx.fda_mean_state(w[:, :d], w0, xg, ALL, mean)
        for variant in (0, 1):
            e = ctx.fda_combine_estimate(mean.view(1, -1), 1, variant, 0.06, 1e-3, buf).as_dict()
            r = oracle.combine(ora, l, m, variant, 0.06, 1e-3)
            assert abs(e["mean_sq"] - r["mean_sq"]) <= REL * r["mean_sq"]
            assert abs(e["est"] - r["est"]) <= 4 * REL * max(r["est"], ubar_sq)
            tol = mean_estimate_tolerance(r, ubar_sq)
            assert abs(e["H"] - r["H"]) <= tol
            check_trigger(e, r, 1e-3, tol)


# ------------------------------------------------------------------- combine / trigger
def test_combine_matches_oracle_on_gpu_states(env):
    torch, oracle, F = env
    rng = np.random.default_rng(21)
    for (K, l, m) in ((5, 5, 250), (60, 7, 500), (3, 4, 33), (1, 1, 1), (7, 16, 64), (9, 6, 1000)):
        slen = 2 + l * m
        st = rng.normal(0, 1e-2, size=(K, slen)).astype(np.float32)
        st[:, 0] = rng.uniform(0.5, 2.0, size=K)
        coeffs = rand_coeffs(rng, l)
        with F.FdaContext(l, m, coeffs, d_max=64, K_max=K) as ctx:
            dev = torch.from_numpy(st).cuda()
            buf = ctx.new_estimate_buffer()
            for variant in (0, 1):
                for eps in (0.0, 0.06):
                    ref0 = oracle.combine(st, l, m, variant, eps, 0.0)
                    for theta in (0.0, 1e-2, float(np.float32(ref0["H"])), 10.0, -1.0):
                        ref = oracle.combine(st, l, m, variant, eps, float(np.float32(theta)))
                        got = ctx.fda_combine_estimate(dev, K, variant, eps, theta, buf).as_dict()
                        tol = check_estimate(got, ref, l)
                        check_trigger(got, ref, theta, tol)
                        assert got["theta"] == np.float32(theta)
                        # the device copy holds the same record
                        raw = bytes(buf.cpu().numpy())
                        assert F.Estimate.from_buffer_copy(raw).H == got["H"]


def test_combine_strict_threshold(env):
    """H exactly representable and equal to Theta: no trigger (Algorithm 1 uses '>')."""
    torch, oracle, F = env
    st = np.zeros((2, 2), dtype=np.float32)
    st[:, 0] = [10.0, 14.0]
    st[:, 1] = [1.0, 3.0]            # H_linear = 12 - 4 = 8
    with F.FdaContext(0, 0, None, d_max=8, K_max=2) as ctx:
        dev, buf = torch.from_numpy(st).cuda(), ctx.new_estimate_buffer()
        e = ctx.fda_combine_estimate(dev, 2, 0, 0.0, 8.0, buf)
        assert e.H == 8.0 and e.trigger == 0
        assert ctx.fda_combine_estimate(dev, 2, 0, 0.0, float(np.nextafter(np.float32(8), 0)), buf).trigger == 1
        assert ctx.fda_combine_estimate(dev, 2, 0, 0.0, 0.0, buf).trigger == 1     # Theta = 0: Synchronous


# ------------------------------------------------------------------------------ average
def test_average_exact_cases_and_gating(env):
    torch, oracle, F = env
    rng = np.random.default_rng(31)
    with F.FdaContext(0, 0, None, d_max=100_000, K_max=64) as ctx:
        buf = ctx.new_estimate_buffer()
        for K, d in ((1, 77), (4, 10_001), (8, 4_096), (16, 3), (64, 999)):
            stride = S.row_stride(d)
            w_np = np.zeros((K, stride), dtype=np.float32)
            w_np[:, :d] = rng.integers(-64, 65, size=(K, d))
            exact = oracle.average(w_np[:, :d])
            for flags in (F.FDA_AVG_UNCONDITIONAL, F.FDA_AVG_UNCONDITIONAL | F.FDA_AVG_BROADCAST):
                w = torch.from_numpy(w_np).cuda()
                w0 = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
                ctx.fda_average_models(w[:, :d], w0, None, flags)
                torch.cuda.synchronize()
                assert np.array_equal(w0.cpu().numpy().astype(np.float64), exact)   # exact in any order
                rows = w.cpu().numpy()
                if flags & F.FDA_AVG_BROADCAST:
                    assert all(np.array_equal(rows[k, :d].astype(np.float64), exact) for k in range(K))
                else:
                    assert np.array_equal(rows, w_np)
                assert not rows[:, d:].any()                   # padding untouched
        # gating by the device-side trigger
        K, d = 4, 5_000
        w_np = rng.normal(size=(K, S.row_stride(d))).astype(np.float32)
        states = torch.zeros((K, 2), dtype=torch.float32, device="cuda")
        states[:, 0] = 1.0
        for theta, fires in ((2.0, False), (0.5, True)):
            est = ctx.fda_combine_estimate(states, K, 0, 0.0, theta, buf)
            assert bool(est.trigger) == fires
            w = torch.from_numpy(w_np).cuda()
            w0 = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
            ctx.fda_average_models(w[:, :d], w0, buf, F.FDA_AVG_BROADCAST)
            torch.cuda.synchronize()
            if fires:
                check_average(w0.cpu().numpy(), oracle.average(w_np[:, :d]))
                assert np.array_equal(w.cpu().numpy()[2, :d], w0.cpu().numpy())
            else:
                assert np.all(w0.cpu().numpy() == 7.0) and np.array_equal(w.cpu().numpy(), w_np)


def test_average_random_and_unaligned(env):
    torch, oracle, F = env
    rng = np.random.default_rng(32)
    with F.FdaContext(0, 0, None, d_max=100_000, K_max=64) as ctx:
        for K, d, stride, off in ((5, 61_706, 61_706, 0), (10, 9_999, 10_001, 1), (60, 20_001, 20_032, 0),
                                  (30, 7, 9, 3)):
            w_np = np.zeros((K, stride), dtype=np.float32)
            w_np[:, :d] = rng.normal(0, 0.05, size=(K, d))
            buf = torch.zeros(K * stride + 8, dtype=torch.float32, device="cuda")
            w = buf[off:off + K * stride].view(K, stride)
            w.copy_(torch.from_numpy(w_np))
            w0buf = torch.zeros(d + 8, dtype=torch.float32, device="cuda")
            w0 = w0buf[off:off + d]
            ctx.fda_average_models(w[:, :d], w0, None, F.FDA_AVG_BROADCAST)
            torch.cuda.synchronize()
            ref = oracle.average(w_np[:, :d])
            check_average(w0.cpu().numpy(), ref)
            got = w.cpu().numpy()
            assert all(np.array_equal(got[k, :d], w0.cpu().numpy()) for k in range(K))
            assert np.array_equal(got[:, d:], w_np[:, d:])


def test_average_with_direction_refresh(env):
    """fda_average_models_xi: the average as before plus xi = (w-bar_new - w_t0_old)/||.||."""
    torch, oracle, F = env
    rng = np.random.default_rng(33)
    with F.FdaContext(0, 0, None, d_max=400_000, K_max=64) as ctx:
        buf = ctx.new_estimate_buffer()
        for K, d, off in ((5, 61_706, 0), (8, 300_001, 0), (60, 20_001, 0), (3, 9, 1)):
            stride = S.row_stride(d) + (1 if off else 0)
            w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
            w_np = np.zeros((K, stride), dtype=np.float32)
            w_np[:, :d] = w_t0 + rng.normal(3e-4, 1e-3, size=(K, d)).astype(np.float32)
            ref_avg = oracle.average(w_np[:, :d])
            ref_xi = oracle.direction(ref_avg, w_t0)
            w = torch.from_numpy(w_np).cuda()
            w0 = torch.from_numpy(w_t0).cuda()
            xi = torch.full((d + 4,), 9.0, dtype=torch.float32, device="cuda")[off:off + d]
            ctx.fda_average_models_xi(w[:, :d], w0, xi, None, F.FDA_AVG_BROADCAST | F.FDA_AVG_UNCONDITIONAL)
            torch.cuda.synchronize()
            check_average(w0.cpu().numpy(), ref_avg)
            got = xi.cpu().numpy().astype(np.float64)
            # the step is a difference of nearby numbers, so xi inherits the fp32 rounding of w-bar
            # (K sequential adds: at most (K/2 + 2) * 2^-24 |w-bar|) amplified by 1/||step||
            step_norm = np.linalg.norm(ref_avg - w_t0)
            tol = (REL * np.maximum(np.abs(ref_xi), 1.0 / np.sqrt(d)) +
                   (K / 2 + 2) * 2.0 ** -24 * np.maximum(np.abs(ref_avg), np.abs(w_t0)) / step_norm)
            assert np.all(np.abs(got - ref_xi) <= tol)
            assert abs(float(np.sum(got * got)) - 1.0) <= 1e-5
            assert all(np.array_equal(w.cpu().numpy()[k, :d], w0.cpu().numpy()) for k in range(K))
        # gate closed: nothing is written; zero step: xi becomes 0
        K, d = 4, 1000
        w = torch.ones((K, d), dtype=torch.float32, device="cuda")
        w0 = torch.ones(d, dtype=torch.float32, device="cuda")
        xi = torch.full((d,), 9.0, dtype=torch.float32, device="cuda")
        st = torch.zeros((K, 2), dtype=torch.float32, device="cuda")
        assert ctx.fda_combine_estimate(st, K, 0, 0.0, 1.0, buf).trigger == 0
        ctx.fda_average_models_xi(w, w0, xi, buf, F.FDA_AVG_BROADCAST)
        torch.cuda.synchronize()
        assert bool((xi == 9.0).all())
        ctx.fda_average_models_xi(w, w0, xi, None, F.FDA_AVG_UNCONDITIONAL)
        torch.cuda.synchronize()
        assert not bool(xi.any())


# ----------------------------------------------------------------- the five workloads
def full_round(env, idx):
    """local state -> combine (both variants, every Theta) -> averaged state -> average, every worker
    and every weight against the oracle (all host cores: about 10 s at the two largest workloads)."""
    torch, oracle, F = env
    wl = S.WORKLOADS[idx]
    w_t0 = S.last_global_model(wl)
    wbuf = S.worker_models(wl, w_t0, threads=16)
    xi = S.unit_direction(wl)
    coeffs = S.hash_coefficients(wl.seed, wl.l)
    d, K = wl.d, wl.K
    ks = list(range(K))
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, wl.l, wl.m, threads=HOST_CORES)
    with F.FdaContext(wl.l, wl.m, coeffs, d_max=d, K_max=K) as ctx:
        w = torch.from_numpy(wbuf).cuda()
        w0 = torch.from_numpy(w_t0).cuda()
        xg = torch.from_numpy(xi).cuda()
        st = torch.empty((K, ctx.state_len), dtype=torch.float32, device="cuda")
        buf = ctx.new_estimate_buffer()
        ctx.fda_local_state(w[:, :d], w0, xg, ALL, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
        worst = check_states(got, ora, wl.l, wl.m, d, rows=ks)
        # combine: the oracle runs on the GPU's own fp32 states (isolates this step) ...
        results = {}
        for variant in (F.FDA_VARIANT_LINEAR, F.FDA_VARIANT_SKETCH):
            for theta in wl.thetas:
                ref = oracle.combine(got, wl.l, wl.m, variant, wl.epsilon, float(np.float32(theta)))
                e = ctx.fda_combine_estimate(st, K, variant, np.float32(wl.epsilon), theta, buf).as_dict()
                tol = check_estimate(e, ref, wl.l)
                check_trigger(e, ref, theta, tol)
                results[(variant, theta)] = e
                # ... and on the oracle's own states, end to end
                ref2 = oracle.combine(ora, wl.l, wl.m, variant, wl.epsilon, float(np.float32(theta)))
                tol2 = check_estimate(e, ref2, wl.l)
                check_trigger(e, ref2, theta, tol2)
        # the one-pass averaged state against the mean of the oracle's K states (linearity)
        mean = torch.empty((ctx.state_len,), dtype=torch.float32, device="cuda")
        ctx.fda_mean_state(w[:, :d], w0, xg, ALL, mean)
        torch.cuda.synchronize()
        _, _, ubar_sq = oracle.variance(wbuf[:, :d], w_t0)
        worst["mean_state"] = check_mean_state(mean.cpu().numpy(), ora, ubar_sq, wl.l, wl.m, d, K)
        e_mean = ctx.fda_combine_estimate(mean.view(1, -1), 1, F.FDA_VARIANT_SKETCH, np.float32(wl.epsilon),
                                          wl.thetas[-1], buf).as_dict()
        e_ref = oracle.combine(ora, wl.l, wl.m, F.FDA_VARIANT_SKETCH, wl.epsilon, float(np.float32(wl.thetas[-1])))
        tol_m = mean_estimate_tolerance(e_ref, ubar_sq)
        assert abs(e_mean["H"] - e_ref["H"]) <= tol_m
        check_trigger(e_mean, e_ref, wl.thetas[-1], tol_m)
        # average (gated by the last sketch estimate, which fires on every workload)
        e = ctx.fda_combine_estimate(st, K, F.FDA_VARIANT_SKETCH, np.float32(wl.epsilon), wl.thetas[-1], buf)
        assert e.trigger == 1
        ctx.fda_average_models(w[:, :d], w0, buf, F.FDA_AVG_BROADCAST)
        torch.cuda.synchronize()
        new_w0 = w0.cpu().numpy()
        check_average(new_w0, oracle.average(wbuf[:, :d]))
        # in-place sync: every row equals the new global model; padding untouched
        for k in (0, K // 2, K - 1):
            assert torch.equal(w[k, :d], w0)
        assert not bool(w[:, d:].any())
        # after synchronisation the variance is zero: all states vanish and nothing fires
        ctx.fda_local_state(w[:, :d], w0, xg, ALL, st)
        e = ctx.fda_combine_estimate(st, K, F.FDA_VARIANT_SKETCH, np.float32(wl.epsilon), 0.0, buf)
        assert not bool(st.any()) and e.H == 0.0 and e.trigger == 0
    return worst, results


def test_workload_1_lenet5(env):
    full_round(env, 1)


def test_workload_2_smallcnn_both_variants(env):
    _, res = full_round(env, 2)
    assert res[(0, 1e-2)]["H"] >= res[(1, 1e-2)]["H"] * 0.9     # linear over-estimates more


def test_workload_3_densenet121_full_round(env):
    full_round(env, 3)


def test_workload_4_densenet201_full_size(env):
    full_round(env, 4)


def test_workload_5_convnextlarge_full_size(env):
    full_round(env, 5)


@pytest.mark.parametrize("l,m", [(3, 100), (8, 1000), (5, 250)])
def test_vgg16_sized_shape_with_other_sketch_sizes(env, l, m):
    """A second workload shape: d = 2.6M (the paper's VGG16* row of Table 2), K = 20, smaller and
    larger sketches than the recommended 5 x 250 (Section 3.3 leaves other sizes open)."""
    torch, oracle, F = env
    wl = S.small_workload(seed=11, d=2_600_000, K=20, l=l, m=m, drift="shared", sigma=1e-3,
                          epsilon=0.06 * (250.0 / m) ** 0.5)
    w_t0 = S.last_global_model(wl)
    wbuf = S.worker_models(wl, w_t0, threads=16)
    xi = S.unit_direction(wl)
    coeffs = S.hash_coefficients(wl.seed, l)
    d, K = wl.d, wl.K
    ks = [0, 9, 19]
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, l, m, workers=ks, threads=3)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w, w0, xg, st = gpu_states(torch, F, ctx, wbuf, w_t0, xi)
        ctx.fda_local_state(w[:, :d], w0, xg, ALL, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
        check_states(got, ora, l, m, d, rows=ks)
        buf = ctx.new_estimate_buffer()
        for variant in (0, 1):
            ref = oracle.combine(got, l, m, variant, wl.epsilon, 1e-2)
            e = ctx.fda_combine_estimate(st, K, variant, np.float32(wl.epsilon), 1e-2, buf).as_dict()
            tol = check_estimate(e, ref, l)
            check_trigger(e, ref, 1e-2, tol)
        ctx.fda_average_models(w[:, :d], w0, buf, F.FDA_AVG_BROADCAST)
        torch.cuda.synchronize()
        check_average(w0.cpu().numpy(), oracle.average(wbuf[:, :d]))


def test_largest_supported_dimension(env):
    """d just below 2^31 (the limit of fda_create), ragged, one worker, one sketch row: 64-bit
    offsets, the top of the hash key range and the last partial tile.  The drift is non-zero only
    in three windows (start, middle, end) so that every cell can be traced to a few indices."""
    torch, oracle, F = env
    d, l, m = (1 << 31) - 4097, 1, 250
    rng = np.random.default_rng(99)
    coeffs = rand_coeffs(rng, l)
    w = torch.zeros((1, d), dtype=torch.float32, device="cuda")
    w0 = torch.zeros(d, dtype=torch.float32, device="cuda")
    windows = [(0, 70_001), (d // 2 - 33_333, d // 2 + 33_334), (d - 100_003, d)]
    host = []
    for lo, hi in windows:
        v = rng.normal(0, 1e-3, size=hi - lo).astype(np.float32)
        base = rng.normal(0, 0.05, size=hi - lo).astype(np.float32)
        w[0, lo:hi] = torch.from_numpy(base + v).cuda()
        w0[lo:hi] = torch.from_numpy(base).cuda()
        host.append((lo, hi, (base + v).astype(np.float32), base))
    # oracle on the windows only (the rest contributes exactly zero): same sums, hash keys offset
    norm, sk = 0.0, np.zeros(m)
    for lo, hi, wv, bv in host:
        u = wv.astype(np.float64) - bv.astype(np.float64)
        norm += float(np.sum(u * u))
        b, sg = oracle.hash_dump(coeffs, l, m, lo, hi - lo)
        np.add.at(sk, b[0], sg[0] * u)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=1) as ctx:
        st = torch.empty((1, ctx.state_len), dtype=torch.float32, device="cuda")
        ctx.fda_local_state(w, w0, None, 1 | 4, st)
        mean = torch.empty(ctx.state_len, dtype=torch.float32, device="cuda")
        ctx.fda_mean_state(w, w0, None, 1 | 4, mean)
        torch.cuda.synchronize()
        ref = np.concatenate([[norm, 0.0], sk])[None]
        check_states(st.cpu().numpy(), ref, l, m, d)
        check_states(mean.cpu().numpy()[None], ref, l, m, d)
        ctx.fda_average_models(w, w0, None, F.FDA_AVG_UNCONDITIONAL)       # K = 1: w_t0 becomes w bit for bit
        torch.cuda.synchronize()
        for lo, hi, wv, _ in host:
            assert np.array_equal(w0[lo:hi].cpu().numpy(), wv)
        assert float(w0[70_001:d // 2 - 33_333].abs().max()) == 0.0


# ------------------------------------------------------------------ host entry point
def test_round_host_matches_device_path(env):
    torch, oracle, F = env
    wl = S.small_workload(seed=9, d=300_007, K=6)
    w_t0 = S.last_global_model(wl)
    wbuf = S.worker_models(wl, w_t0)
    xi = S.unit_direction(wl)
    coeffs = S.hash_coefficients(wl.seed, wl.l)
    d, K = wl.d, wl.K
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, wl.l, wl.m, threads=4)
    ref = oracle.combine(ora, wl.l, wl.m, 1, wl.epsilon, 1e-3)
    avg = oracle.average(wbuf[:, :d])
    with F.FdaContext(wl.l, wl.m, coeffs, d_max=d, K_max=K) as ctx:
        for pinned in (False, True):
            wh = torch.from_numpy(wbuf.copy())
            w0h = torch.from_numpy(w_t0.copy())
            xih = torch.from_numpy(xi.copy())
            sth = torch.empty((K, ctx.state_len), dtype=torch.float32)
            if pinned:
                wh, w0h, xih, sth = wh.pin_memory(), w0h.pin_memory(), xih.pin_memory(), sth.pin_memory()
            e = ctx.fda_round_host(wh[:, :d], w0h, xih, ALL, 1, np.float32(wl.epsilon), 1e-3,
                                   F.FDA_AVG_BROADCAST, sth).as_dict()
            check_states(sth.numpy(), ora, wl.l, wl.m, d)
            tol = check_estimate(e, ref, wl.l)
            check_trigger(e, ref, 1e-3, tol)
            assert e["trigger"]
            check_average(w0h.numpy(), avg)
            assert all(np.array_equal(wh.numpy()[k, :d], w0h.numpy()) for k in range(K))
            # no trigger: host buffers stay as they were
            wh2, w0h2 = torch.from_numpy(wbuf.copy()), torch.from_numpy(w_t0.copy())
            e2 = ctx.fda_round_host(wh2[:, :d], w0h2, xih, ALL, 1, np.float32(wl.epsilon), 1e9,
                                    F.FDA_AVG_BROADCAST, None)
            assert e2.trigger == 0 and np.array_equal(wh2.numpy(), wbuf) and np.array_equal(w0h2.numpy(), w_t0)


# ---------------------------------------------------------------------- error paths
def test_invalid_arguments_are_rejected_on_the_host(env):
    torch, oracle, F = env
    rng = np.random.default_rng(41)
    coeffs = rand_coeffs(rng, 5)
    bad = coeffs.copy(); bad[0] = 0
    for args in ((5, 250, bad, 100, 2), (17, 250, np.ones(6 * 17, np.uint64), 100, 2), (5, 0, coeffs, 100, 2),
                 (5, 40000, coeffs, 100, 2), (5, 250, coeffs, 0, 2), (5, 250, coeffs, 1 << 31, 2),
                 (5, 250, coeffs, 100, 0)):
        with pytest.raises(F.FdaError) as ei:
            F.FdaContext(*args)
        assert ei.value.status == 1
    with pytest.raises(F.FdaError) as ei:          # 16 x 32768 bins cannot fit shared memory
        F.FdaContext(16, 32768, rand_coeffs(rng, 16), 100, 2).close()
    assert ei.value.status == 2
    with F.FdaContext(5, 250, coeffs, d_max=1000, K_max=4) as ctx:
        w = torch.zeros((4, 1024), dtype=torch.float32, device="cuda")
        w0 = torch.zeros(1000, dtype=torch.float32, device="cuda")
        st = torch.zeros((4, ctx.state_len), dtype=torch.float32, device="cuda")
        buf = ctx.new_estimate_buffer()
        big = torch.zeros((5, 1024), dtype=torch.float32, device="cuda")
        for call in (lambda: ctx.fda_local_state(big[:, :1000], w0, None, ALL, st),        # K > K_max
                     lambda: ctx.fda_local_state(w[:, :1000], w0, None, 8, st),            # unknown flag
                     lambda: ctx.fda_local_state(w[:, :1000], None, None, ALL, st),        # null
                     lambda: ctx.fda_combine_estimate(st, 4, 2, 0.0, 1.0, buf),            # bad variant
                     lambda: ctx.fda_combine_estimate(st, 4, 1, -1.0, 1.0, buf),           # eps <= -1
                     lambda: ctx.fda_combine_estimate(st, 4, 1, 0.0, float("nan"), buf),   # theta NaN
                     lambda: ctx.fda_combine_estimate(st, 9, 1, 0.0, 1.0, buf),            # K > K_max
                     lambda: ctx.fda_average_models(w[:, :1000], w0, buf, 4),              # unknown flag
                     lambda: ctx.fda_average_models(w[:, :1000], None, buf, 0)):           # null
            with pytest.raises(F.FdaError) as ei:
                call()
            assert ei.value.status == 1 and ctx.fda_last_error()
        # the context is still usable after rejected calls
        ctx.fda_local_state(w[:, :1000], w0, None, ALL, st)
        torch.cuda.synchronize()
        assert not bool(st.any())
    with F.FdaContext(0, 0, None, d_max=1000, K_max=4) as ctx0:
        st2 = torch.zeros((4, 2), dtype=torch.float32, device="cuda")
        with pytest.raises(F.FdaError):
            ctx0.fda_local_state(w[:, :1000], w0, None, ALL, st2)          # sketch flag, no sketch
        with pytest.raises(F.FdaError):
            ctx0.fda_combine_estimate(st2, 4, 1, 0.0, 1.0, ctx0.new_estimate_buffer())


def test_repeat_runs_agree_within_tolerance(env):
    """Shared-memory atomics make the add order vary between runs: results may differ in the
    last bits but must stay inside the tolerance of each other."""
    a, ref = run_case(env, 8, 50_001, 5, 250, seed=99)
    b, _ = run_case(env, 8, 50_001, 5, 250, seed=99)
    check_states(b, ref, 5, 250, 50_001)
    assert np.allclose(a, b, rtol=1e-4, atol=1e-7)


@pytest.mark.parametrize("n,offset", [(1, 0), (3, 1), (1000, 1), (5_000_003, 3), (1 << 22, 0)])
def test_read_probe_returns_the_sum(env, n, offset):
    """The bandwidth probe is not part of the method; its result is the plain sum (fp64 here)."""
    torch, _, F = env
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n + offset).astype(np.float32)
    buf = torch.from_numpy(x).cuda()
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    with F.FdaContext(0, 0, None, d_max=1024, K_max=1) as ctx:
        ctx.fda_debug_read_probe(buf[offset:], out)
        torch.cuda.synchronize()
        with pytest.raises(F.FdaError):
            ctx.fda_debug_read_probe(buf[:0], out)
    want = x[offset:].astype(np.float64).sum()
    assert abs(float(out.item()) - want) <= 1e-5 * np.abs(x[offset:]).astype(np.float64).sum() + 1e-6


def test_one_context_serves_changing_shapes_and_buffers(env):
    """A context created for (d_max, K_max) is then called with smaller and different shapes and
    with fresh buffers; state that the library keeps between calls (cached tensor maps, partial
    buffers, the combine ticket) must not leak from one call into the next."""
    torch, oracle, F = env
    rng = np.random.default_rng(2024)
    l, m = 5, 250
    coeffs = rand_coeffs(rng, l)
    shapes = [(8, 33_001), (5, 4_099), (8, 33_001), (16, 50_000), (3, 777), (8, 33_001)]
    keep = []                                  # keep earlier buffers alive: new calls get new addresses
    with F.FdaContext(l, m, coeffs, d_max=50_000, K_max=16) as ctx:
        buf = ctx.new_estimate_buffer()
        for K, d in shapes:
            stride = S.row_stride(d)
            w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
            wbuf = np.zeros((K, stride), dtype=np.float32)
            wbuf[:, :d] = w_t0 + rng.normal(0, 1e-3, size=(K, d)).astype(np.float32)
            xi = rng.normal(size=d)
            xi = (xi / np.linalg.norm(xi)).astype(np.float32)
            w, w0, xg, st = gpu_states(torch, F, ctx, wbuf, w_t0, xi)
            keep.append((w, w0, xg, st))
            for _ in range(2):                 # the second call reuses the cached tensor maps
                st.fill_(float("nan"))
                ctx.fda_local_state(w[:, :d], w0, xg, ALL, st)
                torch.cuda.synchronize()
                got = st.cpu().numpy()
                ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, l, m)
                check_states(got, ora, l, m, d)
            for variant in (0, 1):
                ref = oracle.combine(got, l, m, variant, 0.06, 1e-3)
                e = ctx.fda_combine_estimate(st, K, variant, np.float32(0.06), 1e-3, buf).as_dict()
                tol = check_estimate(e, ref, l)
                check_trigger(e, ref, 1e-3, tol)


def _random_case(seed):
    """Seeded random shape: worker count, dimension, sketch size, alignment, pitch, flags."""
    rng = np.random.default_rng(10_000 + seed)
    K = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 48, 64, 70]))
    d = int(rng.choice([1, 2, 5, 31, 127, 128, 129, 1000, 4095, 4096, 4097, 9973, 20_011, 40_009]))
    l, m = [(5, 250), (7, 500), (1, 1), (2, 3), (3, 64), (4, 251), (6, 400), (8, 333), (16, 100), (5, 1000)][
        int(rng.integers(0, 10))]
    misalign = int(rng.choice([0, 0, 0, 1, 2, 3]))
    stride = S.row_stride(d) + int(rng.choice([0, 0, 1, 4, 32]))
    flags = int(rng.choice([7, 7, 7, 5, 4, 6, 3]))
    sigma = float(rng.choice([1e-4, 1e-3, 1e-1]))
    return K, d, l, m, misalign, stride, flags, sigma


@pytest.mark.parametrize("seed", range(36))
def test_local_state_random_shapes(env, seed):
    K, d, l, m, misalign, stride, flags, sigma = _random_case(seed)
    run_case(env, K, d, l, m, seed=seed, flags=flags, misalign=misalign, stride=stride, sigma=sigma)


@pytest.mark.parametrize("seed", range(12))
def test_whole_round_random_shapes(env, seed):
    """Random shape, whole round: states -> estimate (both variants, a threshold on either side
    of the oracle's H) -> gated average with direction refresh -> states after the sync are zero."""
    torch, oracle, F = env
    K, d, l, m, misalign, stride, _, sigma = _random_case(100 + seed)
    rng = np.random.default_rng(500 + seed)
    coeffs = rand_coeffs(rng, l)
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    wbuf = np.zeros((K, stride), dtype=np.float32)
    shared = rng.normal(0, 0.5 * sigma, size=d)
    wbuf[:, :d] = w_t0 + (shared + rng.normal(0, sigma, size=(K, d))).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi, coeffs, l, m)
    eps = 0.06
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        w, w0, xg, st = gpu_states(torch, F, ctx, wbuf, w_t0, xi, ALL, misalign)
        buf = ctx.new_estimate_buffer()
        ctx.fda_local_state(w[:, :d], w0, xg, ALL, st)
        torch.cuda.synchronize()
        got = st.cpu().numpy()
        check_states(got, ora, l, m, d)
        ms = torch.full((ctx.state_len,), float("nan"), dtype=torch.float32, device="cuda")
        ctx.fda_mean_state(w[:, :d], w0, xg, ALL, ms)
        torch.cuda.synchronize()
        ubar = (wbuf[:, :d].astype(np.float64) - w_t0.astype(np.float64)).mean(axis=0)
        check_mean_state(ms.cpu().numpy(), ora, float(ubar @ ubar), l, m, d, K)
        fired = None
        for variant in (0, 1):
            h = oracle.combine(got, l, m, variant, eps, 0.0)["H"]
            for theta in (abs(h) * 2.0 + 1e-30, abs(h) * 0.5):
                ref = oracle.combine(got, l, m, variant, eps, theta)
                e = ctx.fda_combine_estimate(st, K, variant, np.float32(eps), np.float32(theta), buf).as_dict()
                tol = check_estimate(e, ref, l)
                check_trigger(e, ref, theta, tol)
                fired = bool(e["trigger"])
        ref_avg = oracle.average(wbuf[:, :d])
        xi_new = torch.full((d + 4,), 9.0, dtype=torch.float32, device="cuda")[misalign:misalign + d]
        ctx.fda_average_models_xi(w[:, :d], w0, xi_new, buf, F.FDA_AVG_BROADCAST)
        torch.cuda.synchronize()
        if fired:
            check_average(w0.cpu().numpy(), ref_avg)
            assert all(np.array_equal(w.cpu().numpy()[k, :d], w0.cpu().numpy()) for k in range(K))
            ctx.fda_local_state(w[:, :d], w0, xi_new, ALL, st)
            torch.cuda.synchronize()
            assert not st.cpu().numpy().any()              # all drifts are zero after the sync
        else:
            assert np.array_equal(w0.cpu().numpy(), w_t0)
            assert bool((xi_new == 9.0).all())
