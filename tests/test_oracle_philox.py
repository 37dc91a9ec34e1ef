"""Pins for the oracle's Philox-4x32-10 (Salmon et al., SC 2011): published
known answers, uniform conversions, stream layout."""
import os

import numpy as np

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def test_known_answers():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for r in rows:
        w = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(np.array([w[0:4]]), (w[4], w[5]))[0]
        assert [int(v) for v in out] == w[6:10]


def test_bijection_on_counters_small_sample():
    # a keyed bijection never maps two counters to one output
    ctr = np.zeros((4096, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(4096)
    out = oracle.philox4x32_10(ctr, (7, 9))
    assert len({tuple(r) for r in out.tolist()}) == 4096


def test_uniform_conversions():
    x = np.array([0, 255, 512, 0xFFFFFFFF], dtype=np.uint32)
    assert list(oracle.uniform_halfopen(x)) == [0.0, 0.0, 2.0 ** -23, 1 - 2.0 ** -24]
    assert list(oracle.uniform_open(x)) == [2.0 ** -24, 2.0 ** -24, 1.5 * 2.0 ** -23, 1 - 2.0 ** -24]
    # both grids are exact in float32
    assert np.array_equal(oracle.uniform_open(x).astype(np.float32).astype(np.float64), oracle.uniform_open(x))


def test_stream_layout_and_moments():
    seed, step = 0x1A27E2, (5 << 32) | 17
    u = oracle.stream_uniforms(seed, step, row=3, stream=0, count=10)
    key = (seed & 0xFFFFFFFF, seed >> 32)
    blk = oracle.philox4x32_10(np.array([[1, 3, 17, (5 << 2) | 0]]), key)[0]
    assert np.array_equal(u[4:8], oracle.uniform_open(blk).astype(np.float32))
    ua = oracle.stream_uniforms(seed, step, row=3, stream=1)
    blk = oracle.philox4x32_10(np.array([[0, 3, 17, (5 << 2) | 1]]), key)[0]
    assert float(ua) == float(oracle.uniform_halfopen(blk[0]))
    big = oracle.stream_uniforms(seed, 0, row=0, stream=0, count=200000).astype(np.float64)
    assert abs(big.mean() - 0.5) < 4 * (1 / 12 / 200000) ** 0.5
    assert abs(big.var() - 1 / 12) < 1e-3
    hist = np.histogram(big, bins=16, range=(0, 1))[0]
    chi2 = ((hist - 12500) ** 2 / 12500).sum()
    assert chi2 < 45    # 15 dof, p ~ 1e-4
