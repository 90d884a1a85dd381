"""Pins of the CPU checker's sampling rule: exact cases with power-of-two weights worked by hand, the
limits that reduce to greedy choice, and the softmax / top-p definition written out in float64."""
import math

import numpy as np
import pytest

from oracle import sample as osmp
from paper_2407_12021_b200 import inputs as gen

T1 = float(np.float32(osmp.LOG2E))     # at this temperature the exponent is the logit difference itself


def test_power_of_two_weights_by_hand():
    q = osmp.weights([0, -1, -2, -3], T1)
    assert q.tolist() == [2 ** 30, 2 ** 29, 2 ** 28, 2 ** 27]
    # shifts: 2^-41 and below leave nothing of the 31-bit mantissa
    assert osmp.weights([5, 5, -25, -26, -200], T1).tolist() == [2 ** 30, 2 ** 30, 1, 0, 0]
    assert osmp.weights([0, -np.inf, -1], T1).tolist() == [2 ** 30, 0, 2 ** 29]
    # top-p 0.5: the first token alone carries 8/15 of the mass
    assert osmp.nucleus(q, 0.5) == [0]
    assert all(osmp.sample([0, -1, -2, -3], T1, 0.5, u) == 0 for u in (0.0, 0.3, 0.999))
    # top-p 0.75: need 45/32, tokens 0 and 1 (mass 3/2); the boundary between them is at u = 2/3
    assert osmp.nucleus(q, 0.75) == [0, 1]
    assert osmp.sample([0, -1, -2, -3], T1, 0.75, 0.6) == 0
    assert osmp.sample([0, -1, -2, -3], T1, 0.75, 0.6666) == 0
    assert osmp.sample([0, -1, -2, -3], T1, 0.75, 0.6667) == 1
    assert osmp.sample([0, -1, -2, -3], T1, 0.75, 0.99) == 1
    # top-p 1: everything; boundaries at 8/15, 12/15, 14/15
    for u, want in ((0.53, 0), (0.54, 1), (0.79, 1), (0.81, 2), (0.93, 2), (0.94, 3)):
        assert osmp.sample([0, -1, -2, -3], T1, 1.0, u) == want
    # the draw walks the nucleus in id order, whatever the weights' order
    assert sorted(osmp.nucleus(osmp.weights([-2, 0, -3, -1], T1), 0.75)) == [1, 3]
    assert osmp.sample([-2, 0, -3, -1], T1, 0.75, 0.1) == 1 and osmp.sample([-2, 0, -3, -1], T1, 0.75, 0.9) == 3
    # equal weights: lowest ids enter the nucleus first
    assert osmp.nucleus(osmp.weights([1, 1, 1, 1], T1), 0.5) == [0, 1]


def test_weights_follow_the_exponential():
    l = gen.normal([4000], 3.0, 5, 1).numpy().astype(np.float32)
    for temp in (0.3, 1.0, 2.5):
        q = osmp.weights(l, temp).astype(np.float64) / 2.0 ** 30
        want = np.exp((l.astype(np.float64) - float(l.max())) / temp)
        # one float32 rounding of the scaled exponent (|t| up to ~60: 4e-6 absolute), the polynomial (1e-7),
        # and the floor to 30 fractional bits
        assert np.all(np.abs(q - want) <= 1e-5 * want + 2.0 ** -30)


def test_limits_reduce_to_greedy():
    l = gen.normal([8, 500], 1.0, 6, 1).numpy().astype(np.float32)
    u = gen.uniform01(8, 6, 2).numpy()
    for i in range(8):
        assert osmp.sample(l[i], 0.01, 1.0, float(u[i])) == int(np.argmax(l[i]))      # cold: all mass on the maximum
        assert osmp.sample(l[i], 1.0, 1e-4, float(u[i])) == int(np.argmax(l[i]))       # tiny nucleus: the maximum alone
    tie = np.zeros(16, dtype=np.float32)
    assert osmp.sample(tie, 1.0, 0.01, 0.99) == 0
    with pytest.raises(ValueError):
        osmp.sample(l[0], 0.0, 1.0, 0.5)
    with pytest.raises(ValueError):
        osmp.sample(l[0], 1.0, 1.0, 1.0)


@pytest.mark.parametrize("seed,temp,top_p", [(1, 0.7, 0.9), (2, 1.0, 1.0), (3, 1.5, 0.6), (4, 0.4, 0.95)])
def test_draws_follow_the_renormalised_nucleus(seed, temp, top_p):
    V, N = 7, 1 << 14
    l = gen.normal([V], 1.5, seed, 3).numpy().astype(np.float32)
    # the definition in float64: softmax(l / temp), tokens by probability, shortest prefix with mass >= top_p
    p = np.exp((l.astype(np.float64) - float(l.max())) / temp)
    p /= p.sum()
    order = np.argsort(-p, kind="stable")
    cum = np.cumsum(p[order])
    k = V if top_p >= 1.0 else int(np.searchsorted(cum, top_p) + 1)
    if top_p < 1.0:
        assert abs(cum[k - 1] - top_p) > 1e-4 and (k == 1 or abs(cum[k - 2] - top_p) > 1e-4), "seed too close to a nucleus edge"
    members = sorted(order[:k].tolist())
    want = np.zeros(V)
    want[members] = p[members] / p[members].sum()
    draws = np.array([osmp.sample(l, temp, top_p, (i + 0.5) / N) for i in range(N)])
    freq = np.bincount(draws, minlength=V) / N
    assert np.max(np.abs(freq - want)) < 2.0 / N + 1e-5
    assert np.all(np.diff(draws) >= 0)          # inverse CDF in id order


def test_rows_helper():
    l = gen.normal([5, 64], 1.0, 9, 1).numpy().astype(np.float32)
    u = gen.uniform01(5, 9, 2).numpy()
    got = osmp.sample_rows(l, 0.8, 0.9, u)
    assert got.tolist() == [osmp.sample(l[i], 0.8, 0.9, float(u[i])) for i in range(5)]
