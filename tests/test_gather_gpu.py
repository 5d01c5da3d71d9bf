"""GPU parity of the sorted-list sketch kernel (k_local_state_gather) against the CPU oracle.

The library picks that kernel whenever the context holds a list schedule (the test asserts
which kernel ran); the cases are shaped to hit its edges: a ragged last tile, d not a multiple of
4, a last worker group with one or three workers, flag subsets, hash coefficients that put every
index of a sketch row into one cell (the cell is cut into many lists and added atomically) or into
cells in strict rotation, and rows that are only 4-byte aligned (32-bit loads).
Tolerances are those of tests/fda_testlib.py (1e-5 relative, scaled for near-zero cells).
"""
import numpy as np
import pytest

import fda_synth as S
from fda_testlib import check_mean_state, check_states

pytestmark = pytest.mark.gpu

P = (1 << 61) - 1
ALL = 1 | 2 | 4
GATHER = "k_local_state_gather"


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


def run(env, K, d, l, m, seed, flags=ALL, misalign=0, coeffs=None, sigma=1e-3, workers=None, expect=GATHER, launches=2):
    torch, oracle, F = env
    rng = np.random.default_rng(seed)
    stride = S.row_stride(d)
    coeffs = rand_coeffs(rng, l) if coeffs is None else coeffs
    w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
    wbuf = np.zeros((K, stride), dtype=np.float32)
    for k in range(K):                       # row by row: keeps the host footprint small
        wbuf[k, :d] = w_t0 + rng.normal(0, sigma, size=d).astype(np.float32)
    xi = rng.normal(size=d)
    xi = (xi / np.linalg.norm(xi)).astype(np.float32)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        buf = torch.zeros(K * stride + 8, dtype=torch.float32, device="cuda")
        w = buf[misalign:misalign + K * stride].view(K, stride)
        w.copy_(torch.from_numpy(wbuf))
        w0 = torch.from_numpy(w_t0).cuda()
        xg = torch.from_numpy(xi).cuda()
        st = torch.full((K, ctx.state_len), float("nan"), dtype=torch.float32, device="cuda")
        ctx.fda_local_state(w[:, :d], w0, xg, flags, st)
        torch.cuda.synchronize()
        name = ctx.fda_debug_last_kernel()
        assert ctx.fda_debug_last_launches() == launches
        got = st.cpu().numpy()
    if expect is not None:
        assert name == expect, name
    else:
        assert name != GATHER, name
    ks = list(range(K)) if workers is None else workers
    ora = oracle.local_state(wbuf[:, :d], w_t0, xi if (flags & 2) else None, coeffs,
                             l if (flags & 4) else 0, m if (flags & 4) else 0, workers=ks, threads=8)
    full = np.zeros((K, 2 + l * m))
    full[:, :ora.shape[1]] = ora
    if not flags & 1:                         # norm slot off: it must be zero; scales come from the oracle norm
        assert not got[:, 0].any()
        norms = oracle.local_state(wbuf[:, :d], w_t0, None, None, 0, 0, workers=ks, threads=8)[:, 0]
        got = got.copy()
        got[:, 0] = norms
        full[:, 0] = norms
    if not flags & 2:
        assert not got[:, 1].any()
    check_states(got, full, l, m, d, rows=ks)
    return got


D_RAGGED = 600_011          # 98 tiles of 6144 indices, the last one holds 4043; not a multiple of 4


def test_ragged_tail_and_partial_worker_group(env):
    run(env, 57, D_RAGGED, 5, 250, seed=11, workers=[0, 7, 8, 31, 55, 56])


@pytest.mark.parametrize("flags", [4, 1 | 4, 2 | 4])
def test_flag_subsets(env, flags):
    run(env, 57, D_RAGGED, 5, 250, seed=12, flags=flags, workers=[3, 56])


@pytest.mark.parametrize("d", [98 * 6144, 98 * 6144 + 1, 99 * 6144 - 1])
def test_tile_boundaries(env, d):
    run(env, 60, d, 5, 250, seed=13, workers=[0, 59])


def test_three_workers_in_one_group(env):
    run(env, 3, 4_900_003, 5, 250, seed=14)


def test_degenerate_and_rotating_buckets(env):
    """Row 0: a = m, so a*j + b is a multiple of m plus b and every index lands in cell b mod m;
    row 1: a = 1, b = 0, so bucket = j mod m; row 2: c3 = 1 and the other sign coefficients zero,
    so the sign is the parity of j^3 = parity of j; the rest random."""
    l, m = 5, 250
    c = rand_coeffs(np.random.default_rng(15), l)
    c[0], c[1] = m, 7
    c[6], c[7] = 1, 0
    c[14], c[15], c[16], c[17] = 1, 0, 0, 0
    got = run(env, 57, D_RAGGED, l, m, seed=15, coeffs=c, workers=[0, 56])
    row0 = got[:, 2:2 + m]
    assert np.count_nonzero(row0[0]) == 1 and row0[0, 7] != 0.0


def test_other_sketch_shapes(env):
    run(env, 57, D_RAGGED, 3, 100, seed=16, workers=[5, 56])      # long lists: most cells are split
    run(env, 57, D_RAGGED, 7, 300, seed=17, workers=[5, 56])


def test_heavy_tails(env):
    torch, oracle, F = env
    # drift with rare large values (the shape of workload 4): short fp32 runs must keep 1e-5
    run(env, 57, D_RAGGED, 5, 250, seed=18, sigma=1e-3, workers=[1])
    run(env, 57, D_RAGGED, 5, 250, seed=19, sigma=3.0, workers=[1])


def test_unaligned_inputs(env):
    """Rows that start at an odd element (4-byte aligned only) take the same kernel: it loads 32 bits at a time."""
    run(env, 57, D_RAGGED, 5, 250, seed=20, misalign=1, workers=[0, 56])


def test_repeat_runs_agree(env):
    a = run(env, 57, D_RAGGED, 5, 250, seed=21, workers=[2])
    b = run(env, 57, D_RAGGED, 5, 250, seed=21, workers=[2])
    scale = np.maximum(np.abs(a), 1e-30)
    assert float(np.max(np.abs(a - b) / scale)) <= 1e-5


def test_last_kernel_names_follow_the_dispatch(env):
    """Sketch requests are served by the list kernel whatever the size and alignment of the job;
    requests without a sketch by the streaming kernel; sketches whose lists would be too short for
    the schedule by the plain-load kernels - and the library says which one ran."""
    torch, oracle, F = env
    rng = np.random.default_rng(22)
    d, K, l, m = 50_000, 4, 5, 250
    coeffs = rand_coeffs(rng, l)
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        assert ctx.fda_debug_last_kernel() == ""
        w = torch.randn((K, d), device="cuda")
        w0 = torch.randn(d, device="cuda")
        st = torch.empty((K, ctx.state_len), device="cuda")
        ctx.fda_local_state(w, w0, None, 1 | 4, st)
        assert ctx.fda_debug_last_kernel() == GATHER
        ctx.fda_local_state(w, w0, None, 1, st)
        assert ctx.fda_debug_last_kernel() == "k_local_state_linear"
        ctx.fda_local_state(w[:, 1:], w0[1:], None, 1 | 4, st)          # rows start at an odd element
        assert ctx.fda_debug_last_kernel() == GATHER
        torch.cuda.synchronize()
    with F.FdaContext(8, 2000, rand_coeffs(rng, 8), d_max=d, K_max=K) as ctx:   # no schedule for this sketch
        st = torch.empty((K, ctx.state_len), device="cuda")
        ctx.fda_local_state(w, w0, None, 1 | 4, st)
        assert ctx.fda_debug_last_kernel() in ("k_local_state", "k_local_state_fast")
        torch.cuda.synchronize()


def test_sixty_workers_seven_by_five_hundred_run_on_the_list_kernel(env):
    """The shape of the 20M-parameter workload (K = 60, sketch 7 x 500: lists of about ten entries,
    fifteen worker groups on nine blocks each), at a size the oracle does in seconds."""
    run(env, 60, 1_500_007, 7, 500, seed=23, workers=[0, 3, 4, 31, 56, 59])
    run(env, 58, 700_001, 7, 500, seed=24, flags=1 | 4, workers=[0, 55, 57])      # last group: two workers


def test_groups_that_do_not_divide_the_sms_use_the_tail_launches(env):
    """Fifteen worker groups on nine blocks each leave SMs idle; on long vectors those get the last
    tiles of every group through two more launches of the kernel (one block per group for the first
    groups, the other groups after them).  Workers of both tail launches, of the last (partial)
    group, and a ragged last tile."""
    run(env, 60, 3_000_017, 7, 500, seed=28, workers=[0, 3, 51, 52, 55, 59], launches=4)
    run(env, 58, 3_100_003, 7, 500, seed=29, flags=1 | 4, workers=[1, 50, 53, 56, 57], launches=4)


def test_a_round_with_tail_launches_can_be_captured_in_a_graph(env):
    """fda_local_state forks to the context's second stream and joins again with events: legal while
    the caller's stream is being captured.  The replayed graph (local state, estimate, average) gives
    the bits of the eager calls - every reduction of the path has a fixed order."""
    torch, oracle, F = env
    rng = np.random.default_rng(30)
    K, d, l, m = 60, 3_000_017, 7, 500
    w_src = (torch.randn((K, d), device="cuda") * 1e-3)
    w0_src = torch.randn(d, device="cuda") * 0.05
    w_src += w0_src
    with F.FdaContext(l, m, rand_coeffs(rng, l), d_max=d, K_max=K) as ctx:
        def round_(w, w0, states, est):
            ctx.fda_local_state(w, w0, None, 1 | 4, states)
            ctx.fda_combine_estimate(states, K, F.FDA_VARIANT_SKETCH, 0.0424, 1e-6, est, want_host=False)
            ctx.fda_average_models(w, w0, est, F.FDA_AVG_BROADCAST)
        w, w0 = w_src.clone(), w0_src.clone()
        st_e = torch.zeros((K, ctx.state_len), device="cuda")
        est_e = ctx.new_estimate_buffer()
        round_(w, w0, st_e, est_e)
        assert ctx.fda_debug_last_launches() == 4
        torch.cuda.synchronize()
        w_e, w0_e = w.clone(), w0.clone()
        w.copy_(w_src); w0.copy_(w0_src)
        st_g = torch.zeros_like(st_e)
        est_g = ctx.new_estimate_buffer()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            round_(w, w0, st_g, est_g)
        for _ in range(2):                      # the captured round, twice, from the same inputs
            w.copy_(w_src); w0.copy_(w0_src); st_g.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(st_g, st_e)
            assert bytes(est_g.cpu().numpy()) == bytes(est_e.cpu().numpy())
            assert torch.equal(w, w_e) and torch.equal(w0, w0_e)
            assert float(w_e[0, 0]) != float(w_src[0, 0])      # the round did synchronise


def test_context_reports_its_footprint_and_the_schedule_can_be_capped(env):
    torch, oracle, F = env
    rng = np.random.default_rng(25)
    d, K, l, m = 1_000_000, 8, 5, 250
    coeffs = rand_coeffs(rng, l)
    w = torch.randn((K, d), device="cuda") * 1e-3
    w0 = torch.zeros(d, device="cuda")
    with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
        info = ctx.fda_context_info()
        assert info["list_kernel"] == 1 and info["tile_indices"] % 1024 == 0 and info["table_bytes"] == 0
        assert 2.0 * l * d < info["schedule_bytes"] < 3.0 * l * d           # about 2.4 bytes per (row, index)
        assert info["device_bytes"] >= info["schedule_bytes"] and info["schedule_dropped_bytes"] == 0
        st = torch.empty((K, ctx.state_len), device="cuda")
        ctx.fda_local_state(w, w0, None, 1 | 4, st)
        assert ctx.fda_debug_last_kernel() == GATHER and ctx.fda_context_info()["table_bytes"] == 0
        mean = torch.empty((ctx.state_len,), device="cuda")
        ctx.fda_mean_state(w, w0, None, 1 | 4, mean)                         # first use builds the 16-bit table
        assert ctx.fda_debug_last_kernel() == "k_mean_model + k_sketch_vector"
        after = ctx.fda_context_info()
        assert after["table_bytes"] >= 2 * l * d and after["other_lazy_bytes"] >= 4 * d
        torch.cuda.synchronize()
        ref = st.cpu().numpy()
    # a cap below the schedule's size, and no schedule at all: the same states from the other kernels
    for limit in (1_000_000, -1):
        with F.FdaContext(l, m, coeffs, d_max=d, K_max=K, schedule_limit_bytes=limit) as ctx:
            info = ctx.fda_context_info()
            assert info["list_kernel"] == 0 and info["schedule_bytes"] == 0
            assert (info["schedule_dropped_bytes"] > 0) == (limit > 0)
            st = torch.empty((K, ctx.state_len), device="cuda")
            ctx.fda_local_state(w, w0, None, 1 | 4, st)
            assert ctx.fda_debug_last_kernel() in ("k_local_state", "k_local_state_fast")
            torch.cuda.synchronize()
            got = st.cpu().numpy()
            n = ref[:, :1]
            scale = np.maximum(np.abs(ref), np.sqrt(n / m))
            assert float(np.max(np.abs(got - ref) / scale)) <= 2e-5        # two fp32 paths, each within 1e-5 of the oracle


def test_averaged_state_routes(env):
    """Which kernels serve fda_mean_state, and what scratch they make the context allocate: a long
    vector with few workers goes through the list kernel in one pass (nothing allocated); a sketch
    too large for lane-private bins gets its cells from the list kernel run on the averaged drifts
    (d floats, no hash table).  Both against the average of the oracle's per-worker states."""
    torch, oracle, F = env
    rng = np.random.default_rng(27)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    for K, d, l, m, want, lazy in [
        (4, 6144 * 8 * n_sm + 13, 5, 250, "k_mean_state_gather", False),
        (20, 300_007, 7, 500, "k_mean_model + k_mean_state_gather", True),
    ]:
        coeffs = rand_coeffs(rng, l)
        w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
        wbuf = w_t0 + rng.normal(2e-4, 1e-3, size=(K, d)).astype(np.float32)
        ora = oracle.local_state(wbuf, w_t0, None, coeffs, l, m, threads=8)
        _, _, ubar_sq = oracle.variance(wbuf, w_t0)
        with F.FdaContext(l, m, coeffs, d_max=d, K_max=K) as ctx:
            assert ctx.fda_context_info()["list_kernel"] == 1
            mean = torch.full((ctx.state_len,), float("nan"), device="cuda")
            ctx.fda_mean_state(torch.from_numpy(wbuf).cuda(), torch.from_numpy(w_t0).cuda(), None, 1 | 4, mean)
            torch.cuda.synchronize()
            assert ctx.fda_debug_last_kernel() == want
            after = ctx.fda_context_info()
            assert after["table_bytes"] == 0
            assert (4 * d <= after["other_lazy_bytes"] < 5 * d) if lazy else after["other_lazy_bytes"] == 0
            check_mean_state(mean.cpu().numpy(), ora, ubar_sq, l, m, d, K)


def test_more_worker_groups_than_the_scratch_holds_are_refused(env):
    """K beyond what the per-block partial sums were sized for: a status, nothing launched."""
    torch, oracle, F = env
    rng = np.random.default_rng(26)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    K, d, l, m = 32 * n_sm + 1, 4096, 2, 16
    with F.FdaContext(l, m, rand_coeffs(rng, l), d_max=d, K_max=K) as ctx:
        w = torch.zeros((K, d), device="cuda")
        st = torch.full((K, ctx.state_len), 7.0, device="cuda")
        with pytest.raises(F.FdaError) as ei:
            ctx.fda_local_state(w, torch.zeros(d, device="cuda"), None, 1 | 4, st)
        assert ei.value.status == 2
        torch.cuda.synchronize()
        assert bool((st == 7.0).all())
