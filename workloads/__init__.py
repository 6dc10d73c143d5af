"""Seeded synthetic inputs for the Parameter-Server quasi-Newton step.

This module only manufactures inputs: Worker parameter vectors theta_k and gradients
g_k = A theta_k - b + noise of a quadratic J = 1/2 theta^T A theta - b^T theta, in the storage
layout ``[m][n]`` (row k = Worker k).  It contains none of the method's arithmetic (no means of
the Workers, no Gram, no eigen-solve, no update) and is the one module that both the tests of the
CPU oracle and the callers of the CUDA library use, so that both sides read the same bits.

Everything is generated in fixed-size column chunks, each from its own ``torch.Generator`` seeded
by (seed, stream, chunk), so a given (config, device type) always yields the same bits whatever the
memory available.  CPU and CUDA generators are different streams: a comparison always generates
once and hands the same bits to both sides.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Iterator, Optional, Tuple

import numpy as np
import torch

CHUNK = 1 << 20  # columns per generation chunk
BASE_SEED = 170905069

# stream identifiers
_S_D, _S_B, _S_THETA0, _S_PERT, _S_NOISE, _S_W, _S_Z, _S_WRITE = range(8)


@dataclasses.dataclass(frozen=True)
class Config:
    """One workload: shape, storage type, generator parameters and the step's hyper-parameters."""
    index: int
    n: int
    m: int
    dtype: str            # "f32" or "bf16" storage of theta and g
    eig_lo: float         # log10 of the smallest eigenvalue of the diagonal part D
    eig_hi: float         # log10 of the largest
    rank: int             # r of the low-rank part W W^T (0 = diagonal A)
    pert: float           # std of theta_k - theta0
    noise: float          # std of the gradient noise
    tau: float
    lam: float
    writes: int = 0       # asynchronous single-Worker Writes (sliding window), 0 = synchronous

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def with_shape(self, n: Optional[int] = None, m: Optional[int] = None) -> "Config":
        return dataclasses.replace(self, n=self.n if n is None else n, m=self.m if m is None else m)


CONFIGS = (
    Config(0, 4096, 8, "f32", -2, 2, 0, 0.1, 1e-3, 1.0, 0.01),
    Config(1, 1 << 20, 16, "f32", -3, 3, 0, 0.05, 1e-3, 1.0, 0.01),
    Config(2, 25_600_000, 32, "f32", -2, 2, 8, 0.01, 1e-4, 0.5, 0.01),
    Config(3, 124_000_000, 8, "bf16", -2, 2, 0, 0.1, 1e-3, 1.0, 0.01, writes=256),
    Config(4, 1 << 28, 64, "bf16", -2, 2, 16, 0.01, 1e-4, 1.0, 0.01),
)
CONFIG1_LAMBDAS = (0.1, 0.01, 0.001)
CONFIG4_M_SWEEP = (8, 16, 32, 64)


def _gen(device, seed: int, stream: int, chunk: int, extra: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(((seed * 1_000_003 + stream * 7_919 + extra * 104_729) * 65_537 + chunk) % (1 << 62))
    return g


def _chunks(n: int) -> Iterator[Tuple[int, int, int]]:
    for c, i0 in enumerate(range(0, n, CHUNK)):
        yield c, i0, min(i0 + CHUNK, n)


def _normal(shape, device, gen) -> torch.Tensor:
    return torch.randn(shape, device=device, dtype=torch.float32, generator=gen)


def _problem_chunk(cfg: Config, device, c: int, cols: int):
    """(D, b, theta0) of the quadratic on one column chunk, fp32."""
    u = torch.rand(cols, device=device, dtype=torch.float32, generator=_gen(device, cfg.seed, _S_D, c))
    D = torch.pow(10.0, cfg.eig_lo + (cfg.eig_hi - cfg.eig_lo) * u)
    b = _normal(cols, device, _gen(device, cfg.seed, _S_B, c))
    theta0 = _normal(cols, device, _gen(device, cfg.seed, _S_THETA0, c))
    return D, b, theta0


def _w_chunk(cfg: Config, device, c: int, cols: int) -> torch.Tensor:
    return _normal((cfg.rank, cols), device, _gen(device, cfg.seed, _S_W, c)) / math.sqrt(cfg.n)


def helmert(m: int, device="cpu") -> torch.Tensor:
    """m x (m-1) matrix with orthonormal columns spanning the complement of the all-ones vector."""
    Q = torch.zeros(m, m - 1, dtype=torch.float64)
    for c in range(1, m):
        Q[:c, c - 1] = 1.0
        Q[c, c - 1] = -float(c)
        Q[:, c - 1] /= math.sqrt(c * (c + 1))
    return Q.to(device)


def gap_spectrum(m: int, lam: float) -> torch.Tensor:
    """m-1 relative singular values, geometric from 1 down to 1e-4, none inside [lam/3, 3 lam]."""
    k = m - 1
    s = np.geomspace(1.0, 1e-4, k) if k > 1 else np.array([1.0])
    s = s.copy()
    lo, hi = lam / 3.0, lam * 3.0
    for i in range(k):
        if lo <= s[i] <= hi:
            s[i] = hi * 1.25 if s[i] >= lam else lo / 1.25
    s[0] = 1.0
    return torch.tensor(np.sort(s)[::-1].copy(), dtype=torch.float64)


def _perturbation(cfg: Config, device, c: int, cols: int, gap_lam: Optional[float], gap_scale: float,
                  top_on_one_worker: bool = False) -> torch.Tensor:
    """theta_k - theta0 on one chunk, [m][cols] fp32.

    Literal recipe: iid N(0, pert^2).  Gap variant: Z diag(s) Q^T with Z iid N(0,1), Q the Helmert
    basis and s = ``gap_spectrum`` -- the singular values of the centred matrices then follow s, which
    leaves a gap around lam * sigma_1 so that the cut-off j is well defined.  The Helmert basis puts the
    largest mode on Workers 0 and 1; ``top_on_one_worker`` reverses the spectrum's order along the basis,
    so that the largest mode is carried by the last Worker alone (against the mean of the others)."""
    if gap_lam is None:
        return cfg.pert * _normal((cfg.m, cols), device, _gen(device, cfg.seed, _S_PERT, c))
    Z = _normal((cfg.m - 1, cols), device, _gen(device, cfg.seed, _S_Z, c)).double()
    s = gap_spectrum(cfg.m, gap_lam).to(device)
    if top_on_one_worker:
        s = torch.flip(s, dims=(0,))
    Q = helmert(cfg.m, device)
    return (gap_scale * (Q * s) @ Z).float()


def generate(cfg: Config, device="cpu", gap_lam: Optional[float] = None, gap_scale: Optional[float] = None,
             out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None,
             top_on_one_worker: bool = False) -> Tuple[torch.Tensor, torch.Tensor]:
    """theta[m][n], g[m][n] in the config's storage dtype on ``device``.

    g_k = D theta_k + W (W^T theta_k) - b + noise, computed in fp32 from the unrounded theta_k, then
    both are rounded (nearest-even) to the storage dtype.  ``gap_lam`` selects the gap variant of the
    perturbation (see ``_perturbation``); ``gap_scale`` is its overall scale (default ``cfg.pert``)."""
    device = torch.device(device)
    n, m = cfg.n, cfg.m
    if out is None:
        theta = torch.empty((m, n), dtype=cfg.torch_dtype, device=device)
        g = torch.empty((m, n), dtype=cfg.torch_dtype, device=device)
    else:
        theta, g = out
    scale = cfg.pert if gap_scale is None else gap_scale
    wt = None
    if cfg.rank > 0:  # first pass: W^T theta_k, r x m, accumulated in fp64
        wt = torch.zeros((cfg.rank, m), dtype=torch.float64, device=device)
        for c, i0, i1 in _chunks(n):
            _, _, theta0 = _problem_chunk(cfg, device, c, i1 - i0)
            th = theta0.unsqueeze(0) + _perturbation(cfg, device, c, i1 - i0, gap_lam, scale, top_on_one_worker)
            wt += (_w_chunk(cfg, device, c, i1 - i0).double() @ th.double().t())
    for c, i0, i1 in _chunks(n):
        cols = i1 - i0
        D, b, theta0 = _problem_chunk(cfg, device, c, cols)
        th = theta0.unsqueeze(0) + _perturbation(cfg, device, c, cols, gap_lam, scale, top_on_one_worker)
        gr = D.unsqueeze(0) * th - b.unsqueeze(0)
        if wt is not None:
            gr += (wt.t().float() @ _w_chunk(cfg, device, c, cols))
        gr += cfg.noise * _normal((m, cols), device, _gen(device, cfg.seed, _S_NOISE, c))
        theta[:, i0:i1] = th.to(cfg.torch_dtype)
        g[:, i0:i1] = gr.to(cfg.torch_dtype)
    return theta, g


def low_rank_products(cfg: Config, device, begin: int, end: int, gap_lam: Optional[float] = None,
                      gap_scale: Optional[float] = None) -> Optional[torch.Tensor]:
    """The part of W^T theta_k (r x m, fp64) that the columns [begin, end) contribute, or None for a diagonal A.
    ``begin`` and ``end`` must be multiples of the generation chunk (or ``end`` = n).  Summed over a partition of
    [0, n) in chunk order this is what ``generate`` forms in its first pass; a process that holds only a slice of
    the columns adds these over the processes before it calls ``generate_slice``."""
    if cfg.rank == 0:
        return None
    device = torch.device(device)
    scale = cfg.pert if gap_scale is None else gap_scale
    wt = torch.zeros((cfg.rank, cfg.m), dtype=torch.float64, device=device)
    for c, i0, i1 in _chunks(cfg.n):
        if i1 <= begin or i0 >= end:
            continue
        if i0 < begin or i1 > end:
            raise ValueError("slice boundaries must fall on generation chunks")
        _, _, theta0 = _problem_chunk(cfg, device, c, i1 - i0)
        th = theta0.unsqueeze(0) + _perturbation(cfg, device, c, i1 - i0, gap_lam, scale)
        wt += (_w_chunk(cfg, device, c, i1 - i0).double() @ th.double().t())
    return wt


def generate_slice(cfg: Config, device, begin: int, end: int, wt: Optional[torch.Tensor],
                   gap_lam: Optional[float] = None, gap_scale: Optional[float] = None):
    """Columns [begin, end) of what ``generate(cfg)`` returns, as theta[m][end-begin], g[m][end-begin], without
    forming the rest: for a process that holds one slice of an n-sharded problem.  ``wt`` is the full W^T theta
    (``low_rank_products`` added over all slices; None for a diagonal A)."""
    device = torch.device(device)
    m = cfg.m
    scale = cfg.pert if gap_scale is None else gap_scale
    theta = torch.empty((m, end - begin), dtype=cfg.torch_dtype, device=device)
    g = torch.empty((m, end - begin), dtype=cfg.torch_dtype, device=device)
    for c, i0, i1 in _chunks(cfg.n):
        if i1 <= begin or i0 >= end:
            continue
        cols = i1 - i0
        D, b, theta0 = _problem_chunk(cfg, device, c, cols)
        th = theta0.unsqueeze(0) + _perturbation(cfg, device, c, cols, gap_lam, scale)
        gr = D.unsqueeze(0) * th - b.unsqueeze(0)
        if wt is not None:
            gr += (wt.t().float() @ _w_chunk(cfg, device, c, cols))
        gr += cfg.noise * _normal((m, cols), device, _gen(device, cfg.seed, _S_NOISE, c))
        lo, hi = max(i0, begin), min(i1, end)
        theta[:, lo - begin:hi - begin] = th[:, lo - i0:hi - i0].to(cfg.torch_dtype)
        g[:, lo - begin:hi - begin] = gr[:, lo - i0:hi - i0].to(cfg.torch_dtype)
    return theta, g


def write_column(cfg: Config, t: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """The (theta, g) pair of the t-th asynchronous single-Worker Write, each [n] in storage dtype.

    Open loop: theta = theta0 + N(0, pert^2), g = A theta - b + N(0, noise^2), independent of earlier
    updates.  Writes 0..m-1 fill the window, Write t >= m replaces the oldest column."""
    device = torch.device(device)
    if cfg.rank:
        raise ValueError("asynchronous Writes use the diagonal quadratic")
    theta = torch.empty(cfg.n, dtype=cfg.torch_dtype, device=device)
    g = torch.empty(cfg.n, dtype=cfg.torch_dtype, device=device)
    for c, i0, i1 in _chunks(cfg.n):
        cols = i1 - i0
        D, b, theta0 = _problem_chunk(cfg, device, c, cols)
        th = theta0 + cfg.pert * _normal(cols, device, _gen(device, cfg.seed, _S_WRITE, c, extra=2 * t + 1))
        gr = D * th - b + cfg.noise * _normal(cols, device, _gen(device, cfg.seed, _S_WRITE, c, extra=2 * t + 2))
        theta[i0:i1] = th.to(cfg.torch_dtype)
        g[i0:i1] = gr.to(cfg.torch_dtype)
    return theta, g


def quadratic_solution_sample(cfg: Config, idx: np.ndarray) -> np.ndarray:
    """A^-1 b at the given columns for a diagonal config (b/D), fp64, CPU generator stream."""
    if cfg.rank:
        raise ValueError("closed form only for the diagonal quadratic")
    out = np.empty(len(idx), dtype=np.float64)
    cache = {}
    for s, i in enumerate(idx):
        c = int(i) // CHUNK
        if c not in cache:
            cols = min(CHUNK, cfg.n - c * CHUNK)
            D, b, _ = _problem_chunk(cfg, torch.device("cpu"), c, cols)
            cache[c] = (D.double().numpy(), b.double().numpy())
        D, b = cache[c]
        out[s] = b[int(i) % CHUNK] / D[int(i) % CHUNK]
    return out


def to_bits(t: torch.Tensor) -> np.ndarray:
    """Storage tensor -> numpy array of the same bits (float32, or uint16 for bf16), on the host."""
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.float32:
        return t.numpy()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    raise TypeError(t.dtype)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of ``to_bits``."""
    if a.dtype == np.float32:
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)
    if a.dtype == np.uint16:
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)
    raise TypeError(a.dtype)


def tile_columns(block: torch.Tensor, n: int) -> torch.Tensor:
    """Repeat the columns of ``block`` ([m][p] or [p]) periodically up to n columns (n need not be a
    multiple of p).  Used to build full-size inputs whose exact result follows from the block's."""
    p = block.shape[-1]
    reps = (n + p - 1) // p
    if block.dim() == 1:
        return block.repeat(reps)[:n].contiguous()
    return block.repeat(1, reps)[:, :n].contiguous()


def period_permutation(p: int, q: int, seed: int, device="cpu") -> torch.Tensor:
    """The column permutation of period q of ``tile_columns_permuted`` (int64, length p)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed((seed * 2_654_435_761 + q * 40_503 + 17) % (1 << 62))
    return torch.randperm(p, generator=gen).to(device)


def tile_columns_permuted(block: torch.Tensor, n: int, seed: int) -> torch.Tensor:
    """Like ``tile_columns``, but every period holds its own seeded permutation of the block's columns:
    column q*p + c of the result is column ``period_permutation(p, q, seed)[c]`` of the block.  Any quantity that
    is a sum over columns is still (n/p) times the block's, while a result per column can be traced back to its
    source column, so a column offset that is a multiple of p no longer goes unnoticed."""
    p = block.shape[-1]
    if n % p:
        raise ValueError("n must be a multiple of the block's width")
    out = torch.empty(block.shape[:-1] + (n,), dtype=block.dtype, device=block.device)
    for q in range(n // p):
        out[..., q * p:(q + 1) * p] = block.index_select(-1, period_permutation(p, q, seed, block.device))
    return out


def repeated_patterns(n: int, m: int, dtype: str, lam: float, device="cpu", scale: float = 0.25,
                      patterns: int = 64, bases=(0.75, -1.25, 2.5, 0.3125)) -> Tuple[torch.Tensor, torch.Tensor]:
    """Inputs whose columns repeat a small set of values, for checks of reduced-precision Gram arithmetic.

    The Workers' deviations take only ``patterns`` distinct column patterns, X_P = scale * (Q diag(s)) Z_P with Q the
    Helmert basis, s = ``gap_spectrum(m, lam)`` and Z_P the rows 1..m-1 of the Sylvester Hadamard matrix of order
    ``patterns`` (entries +-1, orthogonal rows, so the singular values follow s exactly); the common part of a column
    takes the ``len(bases)`` values of ``bases`` in turn.  g_k[i] = bases[i % B] + X_P[k][(i // B) % patterns] and
    theta_k[i] = theta0[i] + X_P[k][..] / 2, rounded to the storage dtype.  Every rounding error of a kernel that
    splits or truncates the deviations is therefore repeated n / (B * patterns) times instead of averaging out over
    the n columns."""
    if patterns & (patterns - 1) or patterns < m:
        raise ValueError("patterns must be a power of two >= m")
    device = torch.device(device)
    idx = torch.arange(patterns, dtype=torch.int64)
    had = torch.tensor([[1.0 - 2.0 * (bin(r & c).count("1") & 1) for c in range(patterns)] for r in range(1, m)],
                       dtype=torch.float64)
    s = gap_spectrum(m, lam)
    XP = (scale * (helmert(m) * s) @ had).to(device)                 # [m][patterns], fp64
    B = len(bases)
    base = torch.tensor(bases, dtype=torch.float64, device=device)
    tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
    theta = torch.empty((m, n), dtype=tdtype, device=device)
    g = torch.empty((m, n), dtype=tdtype, device=device)
    for c, i0, i1 in _chunks(n):
        i = torch.arange(i0, i1, dtype=torch.int64, device=device)
        x = XP[:, (i // B) % patterns]
        theta0 = _normal(i1 - i0, device, _gen(device, BASE_SEED + 99, _S_THETA0, c)).double()
        g[:, i0:i1] = (base[i % B].unsqueeze(0) + x).float().to(tdtype)
        theta[:, i0:i1] = (theta0.unsqueeze(0) + 0.5 * x).float().to(tdtype)
    del idx
    return theta, g
