"""Seeded closed-loop workload: Workers that evaluate a quadratic's gradient around the Server's iterate.

The paper's experiments (Section 3) train small networks and plot the loss against the number of
Server updates for several Worker counts m; they need datasets.  This module stands in for them with
a problem whose optimum is known: J(theta) = 1/2 theta^T A theta - b^T theta with
A = diag(D) + W diag(S) W^T, D in [d_lo, d_hi] (a well-conditioned bulk) and r orthonormal stiff
directions W with eigenvalues S >> d_hi, so that plain gradient descent is limited to a rate below
2 / max(S) while a step that handles the stiff directions by their secant pairs is not.

Only the problem and the Workers live here (parameters, gradients, the objective and its optimum):
none of the Server's arithmetic.  Everything is drawn from ``torch.Generator`` streams seeded by
(seed, stream, step) on the CPU and moved to the requested device, so that a CPU caller and a GPU
caller see the same bits.
"""
from __future__ import annotations

import dataclasses
from typing import Tuple

import torch

_S_D, _S_W, _S_B, _S_EXPLORE, _S_NOISE = range(5)


@dataclasses.dataclass(frozen=True)
class ClosedLoopConfig:
    n: int = 4096
    rank: int = 6             # number of stiff directions
    d_lo: float = 0.5
    d_hi: float = 1.0
    s_lo: float = 10.0        # stiff eigenvalues, geometric from s_lo to s_hi
    s_hi: float = 100.0
    spread0: float = 0.1      # std of the m initial Workers around theta = 0
    spread: float = 0.01      # std of a Worker's exploration around the Server's iterate afterwards
    noise: float = 1e-3       # std of the gradient noise
    seed: int = 170905069 + 100


def _gen(cfg: ClosedLoopConfig, stream: int, step: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(((cfg.seed * 1_000_003 + stream * 7_919) * 65_537 + step) % (1 << 62))
    return g


@dataclasses.dataclass
class Quadratic:
    """A = diag(D) + W diag(S) W^T and b, in fp64 on ``device``; ``theta_star`` = A^-1 b, ``j_star`` = J(theta_star)."""
    cfg: ClosedLoopConfig
    D: torch.Tensor
    W: torch.Tensor           # [n][r], orthonormal columns
    S: torch.Tensor
    b: torch.Tensor
    theta_star: torch.Tensor
    j_star: float

    def gradient(self, theta: torch.Tensor) -> torch.Tensor:
        """A theta - b for theta [n] or [k][n] (fp64)."""
        t = theta.double()
        return self.D * t + ((t @ self.W) * self.S) @ self.W.t() - self.b

    def objective(self, theta: torch.Tensor) -> float:
        t = theta.double()
        return float(0.5 * torch.dot(t, self.gradient(t) + self.b) - torch.dot(self.b, t))

    def gap(self, theta: torch.Tensor) -> float:
        """J(theta) - J(theta_star) >= 0."""
        return self.objective(theta) - self.j_star


def quadratic(cfg: ClosedLoopConfig, device="cpu") -> Quadratic:
    n, r = cfg.n, cfg.rank
    D = cfg.d_lo + (cfg.d_hi - cfg.d_lo) * torch.rand(n, dtype=torch.float64, generator=_gen(cfg, _S_D))
    W, _ = torch.linalg.qr(torch.randn(n, r, dtype=torch.float64, generator=_gen(cfg, _S_W)))
    S = torch.logspace(torch.log10(torch.tensor(cfg.s_lo)).item(), torch.log10(torch.tensor(cfg.s_hi)).item(), r,
                       dtype=torch.float64)
    b = torch.randn(n, dtype=torch.float64, generator=_gen(cfg, _S_B))
    # A^-1 b by the Woodbury identity: A^-1 = D^-1 - D^-1 W (S^-1 + W^T D^-1 W)^-1 W^T D^-1
    Dib = b / D
    DiW = W / D.unsqueeze(1)
    M = torch.diag(1.0 / S) + W.t() @ DiW
    theta_star = Dib - DiW @ torch.linalg.solve(M, W.t() @ Dib)
    q = Quadratic(cfg, D, W, S, b, theta_star, 0.0)
    q.j_star = q.objective(theta_star)
    dev = torch.device(device)
    for name in ("D", "W", "S", "b", "theta_star"):
        setattr(q, name, getattr(q, name).to(dev))
    return q


def worker(q: Quadratic, centre: torch.Tensor, step: int, spread: float,
           dtype: torch.dtype = torch.float32) -> Tuple[torch.Tensor, torch.Tensor]:
    """One Worker's Write at Server step ``step``: theta = centre + N(0, spread^2) rounded to ``dtype``,
    g = A theta - b + N(0, noise^2) evaluated at the ROUNDED theta and rounded to ``dtype``."""
    cfg = q.cfg
    dev = centre.device
    e = torch.randn(cfg.n, dtype=torch.float64, generator=_gen(cfg, _S_EXPLORE, step)).to(dev)
    z = torch.randn(cfg.n, dtype=torch.float64, generator=_gen(cfg, _S_NOISE, step)).to(dev)
    theta = (centre.double() + spread * e).to(dtype)
    g = (q.gradient(theta) + cfg.noise * z).to(dtype)
    return theta, g


def initial_workers(q: Quadratic, m: int, dtype: torch.dtype = torch.float32) -> Tuple[torch.Tensor, torch.Tensor]:
    """theta[m][n], g[m][n]: m Workers spread around theta = 0 (steps -m..-1 of the random streams)."""
    centre = torch.zeros(q.cfg.n, dtype=torch.float64, device=q.D.device)
    cols = [worker(q, centre, -(k + 1), q.cfg.spread0, dtype) for k in range(m)]
    return torch.stack([c[0] for c in cols]).contiguous(), torch.stack([c[1] for c in cols]).contiguous()
