"""The Server step in closed loop on a quadratic with a known optimum (asynchronous window, Section 2).

Stands in for the convergence curves of the paper's Section 3, whose qualitative statements are checked here:
the method converges faster than SGD; convergence improves as the number of Workers m grows; too few
Workers (fewer secant pairs than stiff directions) at a large learning rate diverge, which the paper lists
among the method's limitations.  The CPU test drives the loop with the oracle; the GPU test drives it with the
CUDA library and checks every step against the oracle on the same window.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as W
from workloads import closed_loop as wl

STEPS = 24
TAU, LAM = 1.0, 1e-3


def oracle_loop(q, m, tau, lam, steps):
    theta, g = wl.initial_workers(q, m)
    gaps = []
    for t in range(steps):
        res = oracle.update(W.to_bits(theta), W.to_bits(g), tau, lam)
        centre = torch.from_numpy(res.theta_new)
        gaps.append(q.gap(centre))
        if not gaps[-1] < 1e12:
            break
        s = t % m
        theta[s], g[s] = wl.worker(q, centre, t, q.cfg.spread)
    return gaps


def sgd_rate(q):
    return 1.9 / float(q.S.max() + q.cfg.d_hi)  # just inside the stability limit 2 / lambda_max(A)


def check_claims(gap0, sgd, by_m):
    # SGD creeps: the bulk eigenvalues see a rate of about 0.01
    assert 0.3 * gap0 < sgd[-1] < gap0
    # four Workers give three secant pairs for six stiff directions: no convergence at tau = 1
    assert by_m[4][-1] > sgd[-1] or len(by_m[4]) < STEPS
    # from 8 Workers on the gap falls by orders of magnitude (single steps are noisy: the tail's median is taken)
    tail = {m: float(np.median(by_m[m][-8:])) for m in (8, 16, 32)}
    assert tail[8] < 1e-3 * gap0
    assert tail[16] < 1e-5 * gap0
    assert tail[32] < 1e-5 * gap0
    # and more Workers are better: mean of log(gap) over the whole run
    level = {m: float(np.mean(np.log(by_m[m]))) for m in (8, 16, 32)}
    assert level[32] < level[16] < level[8] < float(np.mean(np.log(sgd)))


def test_closed_loop_oracle():
    q = wl.quadratic(wl.ClosedLoopConfig())
    gap0 = q.gap(torch.zeros(q.cfg.n, dtype=torch.float64))
    assert abs(float(torch.linalg.norm(q.gradient(q.theta_star))) / float(torch.linalg.norm(q.b))) < 1e-10
    sgd = oracle_loop(q, 8, sgd_rate(q), 2.0, STEPS)
    by_m = {m: oracle_loop(q, m, TAU, LAM, STEPS) for m in (4, 8, 16, 32)}
    check_claims(gap0, sgd, by_m)


@pytest.mark.gpu
def test_closed_loop_gpu_against_oracle_every_step():
    from paper_1709_05069_b200 import closed_loop

    assert torch.cuda.is_available()
    q = wl.quadratic(wl.ClosedLoopConfig(), device="cuda")
    gap0 = q.gap(torch.zeros(q.cfg.n, dtype=torch.float64, device="cuda"))
    checked = []

    def on_step(t, theta, g, theta_new, j, sigma):
        ref = oracle.update(W.to_bits(theta), W.to_bits(g), TAU, LAM)
        s1 = ref.sigma[0]
        assert np.max(np.abs(np.array(sigma) - ref.sigma)) <= 1e-5 * s1
        if (np.abs(ref.sigma / s1 - LAM) < 2e-5).any():  # a sigma on the cut-off, within the sigma tolerance: j is open
            return
        assert j == ref.j
        got = theta_new.double().cpu().numpy()
        assert np.linalg.norm(got - ref.theta_new) <= 1e-5 * np.linalg.norm(ref.theta_new)
        checked.append(t)

    sgd = closed_loop.run(q, 8, sgd_rate(q), 2.0, STEPS)
    by_m = {}
    for m in (4, 8, 16, 32):
        by_m[m] = closed_loop.run(q, m, TAU, LAM, STEPS, on_step=on_step if m >= 8 else None)
    assert len(checked) >= 2 * STEPS
    check_claims(gap0, sgd, by_m)


@pytest.mark.gpu
def test_closed_loop_gpu_bf16_storage():
    from paper_1709_05069_b200 import closed_loop

    q = wl.quadratic(wl.ClosedLoopConfig(), device="cuda")
    gap0 = q.gap(torch.zeros(q.cfg.n, dtype=torch.float64, device="cuda"))

    def on_step(t, theta, g, theta_new, j, sigma):
        ref = oracle.update(W.to_bits(theta), W.to_bits(g), TAU, 1e-2)
        if (np.abs(ref.sigma / ref.sigma[0] - 1e-2) < 2e-5).any():
            return
        checked.append(t)
        assert j == ref.j
        got = oracle.storage_to_f64(W.to_bits(theta_new))
        assert np.linalg.norm(got - ref.theta_new) <= 2e-3 * np.linalg.norm(ref.theta_new)

    checked = []
    gaps = closed_loop.run(q, 16, TAU, 1e-2, STEPS, dtype=torch.bfloat16, on_step=on_step)
    assert len(checked) >= STEPS // 2
    # bf16 parameters: the iterate can only be as close to the optimum as its 8-bit mantissa allows
    assert float(np.median(gaps[-8:])) < 1e-3 * gap0
