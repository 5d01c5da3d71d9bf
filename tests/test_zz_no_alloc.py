"""fda_local_state_linear_noalloc against fda_local_state and against the CPU oracle.

The no-allocation entry point serves callers that cannot create a context because they may
not call cudaMalloc where they run (a hook inside a training step whose framework allocator
holds all free memory; an embedder with a fixed memory budget).  Its scratch is one fixed
array inside the library that keeps whatever the previous call left there, so the check
runs two calls in a row on different inputs and compares each with the context-based entry
point and with the oracle's fp64 norm and projection, within the tolerance the other parity
tests use.  Collected last on purpose.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

REL = 1e-5


def _reference(F, torch, w, w0, xi, flags):
    K, d = w.shape
    with F.FdaContext(0, 0, None, d_max=d, K_max=K) as ctx:
        st = torch.empty((K, 2), dtype=torch.float32, device="cuda")
        ctx.fda_local_state(w, w0, xi, flags, st)
        torch.cuda.synchronize()
        return st.cpu().numpy().astype(np.float64)


def test_no_alloc_entry_point_matches_context_entry_point_twice_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    import paper_2405_20988_b200 as F

    rng = np.random.default_rng(2024)
    cases = [(9, 300_007, 1e-3, 1 | 2), (64, 12_345, 5e-3, 1 | 2), (3, 5, 1e-2, 1)]
    outs = []
    for K, d, sigma, flags in cases:                      # back to back, no context in between
        stride = (d + 31) // 32 * 32 + 1                  # odd pitch: rows are not 16-byte aligned
        w_t0 = rng.normal(0, 0.05, size=d).astype(np.float32)
        wbuf = np.zeros((K, stride), dtype=np.float32)
        wbuf[:, :d] = w_t0 + rng.normal(0, sigma, size=(K, d)).astype(np.float32)
        xi = rng.normal(size=d)
        xi = (xi / np.linalg.norm(xi)).astype(np.float32)
        w = torch.from_numpy(wbuf).cuda()[:, :d]
        w0 = torch.from_numpy(w_t0).cuda()
        xg = torch.from_numpy(xi).cuda()
        states = torch.full((K, 2), float("nan"), dtype=torch.float32, device="cuda")
        before = torch.cuda.memory_allocated()
        F.fda_local_state_linear_noalloc(w, w0, xg, flags, states)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before     # the wrapper created no tensor
        outs.append((states.cpu().numpy().astype(np.float64), w, w0, xg, flags, d, wbuf, w_t0, xi))
    import oracle
    for got, w, w0, xg, flags, d, wbuf, w_t0, xi in outs:
        ora = oracle.local_state(wbuf[:, :d], w_t0, xi if flags & 2 else None, None, 0, 0, threads=4)
        for ref in (_reference(F, torch, w, w0, xg, flags), ora):
            n = ref[:, 0]
            assert np.all(np.abs(got[:, 0] - n) <= REL * n)
            scale = np.maximum(np.abs(ref[:, 1]), np.sqrt(n / d))
            assert np.all(np.abs(got[:, 1] - ref[:, 1]) <= REL * scale)
        if not flags & 2:
            assert not got[:, 1].any()
    # beyond the fixed scratch: refused with a clear error, nothing launched
    K = F.FDA_NOALLOC_MAX_WORKERS + 1
    w = torch.zeros((K, 64), dtype=torch.float32, device="cuda")
    st = torch.zeros((K, 2), dtype=torch.float32, device="cuda")
    with pytest.raises(F.FdaError) as ei:
        F.fda_local_state_linear_noalloc(w, torch.zeros(64, device="cuda"), None, 1, st)
    assert ei.value.status == 2 and "FDA_NOALLOC_MAX_WORKERS" in str(ei.value)
