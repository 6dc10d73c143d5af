"""Closed-loop run of the Server step on a quadratic with a known optimum.

Stands in for the convergence curves of the paper's Section 3 (loss against Server updates for several
Worker counts m, with plain SGD beside them), which need datasets: here the Workers evaluate the gradient
of J = 1/2 theta^T A theta - b^T theta (``workloads.closed_loop``) and every Server step runs in the CUDA
library.  Asynchronous mode of Section 2: the Server keeps the m latest (theta, g) pairs; after each update
one Worker evaluates the gradient near theta_new and its Write replaces the oldest pair (``qn_push``), then
``qn_update_window`` gives the next iterate.  ``lam > 1`` keeps no mode (j = 0), which is SGD on the window's
means (the special case the paper notes after Eq. (4)).

    python -m paper_1709_05069_b200.closed_loop [--n 4096] [--steps 40] [--workers 4 8 16 32]
"""
from __future__ import annotations

import argparse
from typing import Callable, List, Optional

import torch

from workloads import closed_loop as wl

from . import qn


def run(q: wl.Quadratic, m: int, tau: float, lam: float, steps: int, dtype: torch.dtype = torch.float32,
        on_step: Optional[Callable] = None, diverged: float = 1e12) -> List[float]:
    """J(theta_t) - J(theta*) after each of ``steps`` Server updates with m Workers.  ``q`` must live on the GPU.

    ``on_step(t, theta_window, g_window, theta_new, j, sigma)`` is called after every update with the window the
    update was computed from (copies, rows in slot order) -- the tests use it to check every step."""
    if not q.D.is_cuda:
        raise ValueError("the problem must be on the GPU: quadratic(cfg, device='cuda')")
    n = q.cfg.n
    gaps: List[float] = []
    theta, g = wl.initial_workers(q, m, dtype)
    theta_new = torch.empty(n, dtype=dtype, device=q.D.device)
    with qn.qn_create(n, m, dtype) as h:
        for k in range(m):
            qn.qn_push(h, -1, theta[k], g[k])
        for t in range(steps):
            j, sigma, _ = qn.qn_update_window(h, tau, lam, theta_new)
            gaps.append(q.gap(theta_new))
            if on_step is not None:
                on_step(t, theta.clone(), g.clone(), theta_new.clone(), j, sigma)
            if not gaps[-1] < diverged:  # also stops on NaN
                break
            s = t % m  # the oldest pair: the initial Workers filled slots 0..m-1 in order
            theta[s], g[s] = wl.worker(q, theta_new, t, q.cfg.spread, dtype)
            qn.qn_push(h, -1, theta[s], g[s])
    return gaps


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--workers", type=int, nargs="+", default=[4, 8, 16, 32])
    ap.add_argument("--tau", type=float, default=1.0)
    ap.add_argument("--lam", type=float, default=1e-3)
    ap.add_argument("--dtype", choices=("f32", "bf16"), default="f32")
    a = ap.parse_args(argv)
    dtype = torch.float32 if a.dtype == "f32" else torch.bfloat16
    q = wl.quadratic(wl.ClosedLoopConfig(n=a.n), device="cuda")
    gap0 = q.gap(torch.zeros(a.n, dtype=torch.float64, device="cuda"))
    tau_sgd = 1.9 / float(q.S.max() + q.cfg.d_hi)
    rows = [("SGD, m = 8, tau = %.4f" % tau_sgd, run(q, 8, tau_sgd, 2.0, a.steps, dtype))]
    for m in a.workers:
        rows.append(("m = %d, tau = %g, lambda = %g" % (m, a.tau, a.lam), run(q, m, a.tau, a.lam, a.steps, dtype)))
    print("J(0) - J* = %.4g; J(theta_t) - J* after t Server updates" % gap0)
    marks = [t for t in (1, 2, 5, 10, 20, 40, 80) if t <= a.steps]
    print("%-36s" % "" + "".join("%12s" % ("t = %d" % t) for t in marks))
    for name, gaps in rows:
        cells = ["%12.3e" % gaps[t - 1] if t <= len(gaps) else "%12s" % "diverged" for t in marks]
        print("%-36s" % name + "".join(cells))


if __name__ == "__main__":
    main()
