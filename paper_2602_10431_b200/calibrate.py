"""Global threshold for a requested average execution ratio (host control loop).

The paper adjusts the execution ratio after training through one global theta
(Sec. 3.4, Eq. 9) found by a grid search on calibration samples (App. A.1).
This module is the ratio-targeted version of that search: it looks for the
theta at which the average execution ratio R_avg of a calibration batch (executed
(token, layer) pairs over valid tokens x layers) equals a target.  A layer's
scores depend on which tokens the earlier layers executed, hence on theta
itself, so the search iterates: run the stack at theta_i, pool the router scores
of all layers, take their (1 - target) quantile on the device
(qtale_theta_for_ratio) as theta_{i+1}.  Observed (theta, R_avg) pairs bracket the
target; when a quantile step leaves the bracket the loop bisects instead.  All
arithmetic on tensors happens in the library's kernels; this file only compares
two numbers per iteration.
"""
from __future__ import annotations


def search_theta(run, target, tol=0.005, theta0=0.5, max_iters=12):
    """run(theta) -> (r_avg, theta_suggested): executes the calibration batch at theta and
    returns the measured average ratio and the pooled-score quantile for `target`.
    Returns (theta, r_avg, history)."""
    lo = hi = None  # lo: largest theta seen with r_avg above target; hi: smallest with r_avg below
    theta = float(theta0)
    history = []
    best = None
    for _ in range(max_iters):
        r, nxt = run(theta)
        history.append((theta, r))
        if best is None or abs(r - target) < abs(best[1] - target):
            best = (theta, r)
        if abs(r - target) <= tol:
            break
        if r > target:
            lo = theta if lo is None else max(lo, theta)
        else:
            hi = theta if hi is None else min(hi, theta)
        inside = (lo is None or nxt > lo) and (hi is None or nxt < hi)
        if inside and nxt != theta:
            theta = float(nxt)
        elif lo is not None and hi is not None:
            theta = 0.5 * (lo + hi)
        elif lo is not None:       # everything seen executes too much: raise theta
            theta = 0.5 * (lo + 1.0)
        else:
            theta = 0.5 * hi
    return best[0], best[1], history


def calibrate_model_theta(api, mcfg, layers, embed, ids, cu_seqlens, ws, hidden, target,
                          valid=None, tol=0.005, theta0=0.5, max_iters=12):
    """Finds the global theta of a model for a target R_avg on one calibration batch.
    Host reads per iteration: the per-layer executed counts and the suggested theta."""
    import torch
    L = mcfg.n_layers
    T = int(ids.shape[0])
    dev = ids.device
    scores = torch.empty(L, T, dtype=torch.float32, device=dev)
    counts = torch.zeros(L, dtype=torch.int32, device=dev)
    n_valid = T if valid is None else int(valid.sum().item())
    valid_all = None if valid is None else valid.repeat(L).contiguous()
    out = {}

    def run(theta):
        mcfg.layer.select_mode = api.SELECT_THRESHOLD
        mcfg.layer.theta = float(theta)
        api.model_prefill(mcfg, layers, embed, ids, cu_seqlens, ws, hidden, per_layer_n_exec=counts,
                          valid=valid, layer_scores_out=scores)
        th, _ = api.theta_for_ratio(scores.view(-1), target, valid=valid_all, out=out)
        out.setdefault("theta", th)
        r_avg = float(counts.sum().item()) / float(L * max(n_valid, 1))
        return r_avg, float(th.item())

    return search_theta(run, target, tol, theta0, max_iters)
