"""Pins for the oracle's building blocks: random numbers, logarithm, iteration time, length tables, bins."""
import ctypes as C
import math
import os

import numpy as np

from qsim_inputs import lengths as qlen
from qsim_inputs.spec import LMAX

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _philox(L, ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    L.orc_philox4x32_10(c, k, o)
    return list(o)


def test_philox_known_answers(oracle_lib):
    # Published vectors of the generator (SC'11 paper's reference library).
    n = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert _philox(oracle_lib, w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_philox_is_a_bijection_per_key_and_sensitive_to_every_word(oracle_lib):
    base = _philox(oracle_lib, [1, 2, 3, 4], [5, 6])
    seen = {tuple(base)}
    for pos in range(4):
        ctr = [1, 2, 3, 4]
        ctr[pos] ^= 1
        seen.add(tuple(_philox(oracle_lib, ctr, [5, 6])))
    for pos in range(2):
        key = [5, 6]
        key[pos] ^= 1
        seen.add(tuple(_philox(oracle_lib, [1, 2, 3, 4], key)))
    assert len(seen) == 7


def test_philox_words_are_equidistributed(oracle_lib):
    # chi-square of the top byte of each output word over 2^14 consecutive counters
    counts = np.zeros((4, 256), np.int64)
    for i in range(1 << 14):
        for k, w in enumerate(_philox(oracle_lib, [i, 0, 7, 9], [123, 456])):
            counts[k, w >> 24] += 1
    expect = (1 << 14) / 256
    chi2 = ((counts - expect) ** 2 / expect).sum(axis=1)
    assert np.all(chi2 < 400.0)   # 255 dof: mean 255, sd 22.6


def test_u53_range_and_resolution(oracle_lib):
    assert oracle_lib.orc_u53(0, 0) == 2.0 ** -53
    assert oracle_lib.orc_u53(0xFFFFFFFF, 0xFFFFFFFF) == 1.0
    assert oracle_lib.orc_u53(0x80000000, 0) == 0.5 + 2.0 ** -53
    # the low 11 bits of the second word are dropped
    assert oracle_lib.orc_u53(5, 0x7FF) == oracle_lib.orc_u53(5, 0)
    assert oracle_lib.orc_u53(5, 0x800) == oracle_lib.orc_u53(5, 0) + 2.0 ** -53


def test_qlog_matches_libm(oracle_lib):
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.uniform(0.0, 1.0, 20000), 2.0 ** -rng.uniform(0, 53, 20000),
                         [1.0, 0.5, 2.0 ** -53, math.sqrt(0.5), np.nextafter(1.0, 0.0)]])
    xs = xs[xs > 0]
    for x in xs:
        got = oracle_lib.orc_qlog(float(x))
        ref = math.log(float(x))
        assert abs(got - ref) <= 4e-16 * max(1.0, abs(ref)), (x, got, ref)
    assert oracle_lib.orc_qlog(1.0) == 0.0


def test_qlog_exponential_variates_have_unit_mean_and_variance(oracle_lib):
    # E = -qlog(U) must be a unit exponential: mean 1, variance 1 (CLT bands at 5 sigma)
    n = 1 << 15
    e = np.empty(n)
    for i in range(n):
        w = _philox(oracle_lib, [i, 0, 0, 0], [42, 0])
        e[i] = -oracle_lib.orc_qlog(oracle_lib.orc_u53(w[0], w[1]))
    assert abs(e.mean() - 1.0) < 5.0 / math.sqrt(n)
    assert abs(e.var() - 1.0) < 5.0 * math.sqrt(8.0 / n)
    assert e.min() >= 0.0


def test_tau_two_regimes(oracle_lib):
    bench = (C.c_double * 6)(5e-3, 2e-5, 5e-5, 5e-3, 5e-5, 0.0)
    # benchmark law: 5 ms + 0.02 ms * prefill tokens + 0.05 ms * decodes
    assert oracle_lib.orc_tau(bench, 256, 0, 0) == 5e-3 + 2e-5 * 256
    assert abs(oracle_lib.orc_tau(bench, 256, 31, 0) - (0.005 + 0.00512 + 0.00155)) < 1e-18
    assert abs(oracle_lib.orc_tau(bench, 0, 32, 0) - 0.0066) < 1e-18
    paper = (C.c_double * 6)(0.0174, 6.2e-5, 0.0, 0.022, 0.0, 0.0)
    # Eq. (3): tau_mix(C) = alpha + beta C, independent of the decode count; Eq. (2): tau_solo = c
    assert oracle_lib.orc_tau(paper, 256, 0, 0) == oracle_lib.orc_tau(paper, 256, 15, 0) == 0.0174 + 6.2e-5 * 256
    assert oracle_lib.orc_tau(paper, 0, 1, 0) == oracle_lib.orc_tau(paper, 0, 16, 0) == 0.022
    kv = (C.c_double * 6)(0.0174, 6.2e-5, 0.0, 0.0089, 0.0, 1.08e-7)
    # Section 6.1 solo fit: T_solo(K) = 0.0089 + 1.08e-7 K
    assert abs(oracle_lib.orc_tau(kv, 0, 4, 100000) - (0.0089 + 1.08e-7 * 100000)) < 1e-18


def test_table_length_against_searchsorted_and_distribution(oracle_lib):
    tabs = qlen.lognormal_tables([((5.0, 0.5), (7.5, 0.6))])
    rng = np.random.default_rng(1)
    for kind in range(2):
        thr = np.ascontiguousarray(tabs[0, kind])
        ws = np.concatenate([rng.integers(0, 1 << 32, 3000, dtype=np.uint64).astype(np.uint32),
                             np.array([0, 1, 0xFFFFFFFF, thr[0], thr[100], thr[100] - 1], np.uint32)])
        ref = 1 + np.searchsorted(thr[: LMAX - 1], ws, side="right")
        got = [oracle_lib.orc_table_length(thr.ctypes.data_as(C.c_void_p), int(w)) for w in ws]
        assert np.array_equal(np.array(got), ref)
        assert min(got) >= 1 and max(got) <= LMAX
    # the table reproduces round-and-clip lognormal sampling: compare means with direct sampling
    mu, sigma = 5.0, 0.5
    direct = np.clip(np.rint(np.exp(mu + sigma * rng.standard_normal(400000))), 1, LMAX)
    assert abs(qlen.table_mean(tabs[0, 0]) - direct.mean()) < 5 * direct.std() / math.sqrt(direct.size)
    pmf = qlen.table_pmf(tabs[0, 0])
    assert abs(pmf.sum() - 1.0) < 1e-12 and pmf.min() >= 0.0
    # Kolmogorov distance between the table's CDF and the empirical CDF of direct sampling
    emp = np.bincount(direct.astype(np.int64), minlength=LMAX + 1)[1:] / direct.size
    assert np.abs(np.cumsum(emp) - np.cumsum(pmf)).max() < 1.95 / math.sqrt(direct.size) * 1.5


def test_hist_bin_is_log_linear(oracle_lib):
    b = oracle_lib.orc_hist_bin
    assert b(2.0 ** -20) == 0 and b(1e-9) == 0 and b(0.0) == 0
    assert b(2.0 ** -19) == 32 and b(1.0) == 20 * 32 and b(1.5) == 20 * 32 + 16
    assert b(1e9) == 1023
    # monotone, 32 bins per octave
    xs = np.geomspace(1e-6, 4000.0, 5000)
    bins = [b(float(x)) for x in xs]
    assert all(b1 <= b2 for b1, b2 in zip(bins, bins[1:]))
    assert b(0.013) - b(0.0065) == 32
