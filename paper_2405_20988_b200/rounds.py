"""Multi-round driver: Algorithm 1 of the FDA paper with a caller-supplied stand-in for the
local optimiser.  Every step the models drift (``drift_fn``), the local states are formed,
combined into the variance estimate H and, when H > Theta, the models are averaged in place.
All arithmetic of a step runs in libfda; this module only sequences the calls and keeps the
communication account of Section 4 ("communication cost": bytes all workers would transmit -
their local state every step, their model at every synchronisation).
"""
from __future__ import annotations

from .binding import (FDA_AVG_BROADCAST, FDA_STATE_LINEAR, FDA_STATE_NORM, FDA_STATE_SKETCH,
                      FDA_VARIANT_LINEAR, FDA_VARIANT_SKETCH, FdaContext)


def run_rounds(ctx: FdaContext, w, w_t0, xi, steps: int, drift_fn, variant: int, epsilon: float,
               theta: float, refresh_xi: bool = False, averaged_state: bool = False, graph: bool = False):
    """Run ``steps`` steps of Algorithm 1 on device tensors ``w`` (K x d view), ``w_t0`` (d),
    ``xi`` (d or None).  ``drift_fn(t, w)`` must update ``w`` in place (the synthetic
    Optimize).  ``refresh_xi`` re-derives xi from the last two global models at every
    synchronisation (Section 3.2); ``averaged_state`` uses fda_mean_state instead of the K
    per-worker states (same estimate by linearity of the sketch).  ``graph`` captures the library
    calls of a step (state, estimate, the average gated on the device by the trigger word) in a
    CUDA graph after the first step and replays it for the others: one launch per step and no host
    synchronisation until the end, for models small enough that launches dominate a step.

    Returns a dict with the per-step estimates ``H``, the list of synchronisation steps
    ``syncs`` and the bytes that the K workers would have sent: ``state_bytes`` (every step) and
    ``model_bytes`` (every synchronisation)."""
    import torch

    K, d = w.shape
    sketch = variant == FDA_VARIANT_SKETCH
    flags = FDA_STATE_NORM | (FDA_STATE_SKETCH if sketch else FDA_STATE_LINEAR)
    if variant not in (FDA_VARIANT_LINEAR, FDA_VARIANT_SKETCH):
        raise ValueError("variant must be FDA_VARIANT_LINEAR or FDA_VARIANT_SKETCH")
    if refresh_xi and xi is None:
        raise ValueError("refresh_xi needs an xi tensor to write into")
    states = torch.empty((1 if averaged_state else K, ctx.state_len), dtype=torch.float32, device=w.device)
    est_buf = ctx.new_estimate_buffer(w.device)
    per_worker_state = 4 * (1 + (ctx.l * ctx.m if sketch else 1))
    out = {"H": [], "syncs": [], "state_bytes": 0, "model_bytes": 0}

    def library_calls(want_host):
        if averaged_state:
            ctx.fda_mean_state(w, w_t0, None if sketch else xi, flags, states.view(-1))
            est = ctx.fda_combine_estimate(states, 1, variant, epsilon, theta, est_buf, want_host=want_host)
        else:
            ctx.fda_local_state(w, w_t0, None if sketch else xi, flags, states)
            est = ctx.fda_combine_estimate(states, K, variant, epsilon, theta, est_buf, want_host=want_host)
        if want_host and not est.trigger:
            return est
        if refresh_xi:
            ctx.fda_average_models_xi(w, w_t0, xi, est_buf, FDA_AVG_BROADCAST)
        else:
            ctx.fda_average_models(w, w_t0, est_buf, FDA_AVG_BROADCAST)
        return est

    def account(t, H, trigger):
        out["H"].append(float(H))
        out["state_bytes"] += K * per_worker_state
        if trigger:
            out["syncs"].append(t)
            out["model_bytes"] += K * d * 4

    if graph and steps > 1:
        # step 0 eagerly (it also makes the library allocate what it allocates on first use), then
        # the same calls recorded once and replayed; the estimates are read back at the end
        from .binding import Estimate
        drift_fn(0, w)
        est = library_calls(True)
        account(0, est.H, est.trigger)
        history = torch.zeros((steps, est_buf.numel()), dtype=torch.uint8, device=w.device)
        torch.cuda.synchronize(w.device)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            library_calls(False)
        for t in range(1, steps):
            drift_fn(t, w)
            g.replay()
            history[t].copy_(est_buf)
        torch.cuda.synchronize(w.device)
        host = history.cpu().numpy()
        for t in range(1, steps):
            e = Estimate.from_buffer_copy(bytes(host[t]))
            account(t, e.H, e.trigger)
        return out

    for t in range(steps):
        drift_fn(t, w)
        est = library_calls(True)
        account(t, est.H, est.trigger)
    return out
