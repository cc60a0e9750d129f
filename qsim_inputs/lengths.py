"""Integer length tables for lognormal request lengths, built once on the host.

A class's prompt (or output) length is  clip(round(exp(mu + sigma Z)), 1, LMAX).  Its CDF on the
integers is  F(k) = Phi((ln(k + 1/2) - mu) / sigma)  for 1 <= k < LMAX and F(LMAX) = 1.
A simulator maps one uniform 32-bit word w to a length by
    len = 1 + #{ j in [0, LMAX-1) : thr[j] <= w },   thr[j] = round(F(j + 1) * 2^32) (saturated),
so both simulators obtain identical integers from identical words without ever calling exp/log.
"""
from __future__ import annotations

import math

import numpy as np

from .spec import LMAX


def _phi(z: float) -> float:
    return 0.5 * math.erfc(-z / math.sqrt(2.0))


def lognormal_cdf_int(mu: float, sigma: float) -> np.ndarray:
    """F(k) for k = 1..LMAX (index k-1)."""
    F = np.empty(LMAX)
    for k in range(1, LMAX):
        F[k - 1] = _phi((math.log(k + 0.5) - mu) / sigma)
    F[LMAX - 1] = 1.0
    return F


def thresholds_from_cdf(F: np.ndarray) -> np.ndarray:
    """uint32[LMAX]; entry LMAX-1 is padding (0xFFFFFFFF) and is never read."""
    t = np.rint(F[: LMAX - 1] * 4294967296.0)
    t = np.minimum(np.maximum(t, 0.0), 4294967295.0)
    t = np.maximum.accumulate(t)
    out = np.full(LMAX, 0xFFFFFFFF, dtype=np.uint32)
    out[: LMAX - 1] = t.astype(np.uint32)
    return out


def table_pmf(thr: np.ndarray) -> np.ndarray:
    """Exact pmf over lengths 1..LMAX implied by a threshold table (what a simulator samples)."""
    t = thr[: LMAX - 1].astype(np.float64)
    edges = np.concatenate(([0.0], t, [4294967296.0]))
    return np.diff(edges) / 4294967296.0


def table_mean(thr: np.ndarray) -> float:
    return float(np.dot(np.arange(1, LMAX + 1, dtype=np.float64), table_pmf(thr)))


def lognormal_tables(params) -> np.ndarray:
    """params: per class ((mu_in, sigma_in), (mu_out, sigma_out)) -> uint32 [I, 2, LMAX]."""
    out = np.empty((len(params), 2, LMAX), dtype=np.uint32)
    for i, pair in enumerate(params):
        for kind, (mu, sigma) in enumerate(pair):
            out[i, kind] = thresholds_from_cdf(lognormal_cdf_int(mu, sigma))
    return np.ascontiguousarray(out)


def table_mean_chunks(thr: np.ndarray, C: int) -> float:
    """E ceil(len / C): mean number of prefill iterations of a request drawn from the table."""
    k = np.arange(1, LMAX + 1, dtype=np.float64)
    return float(np.dot(np.ceil(k / C), table_pmf(thr)))
