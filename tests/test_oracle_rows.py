"""Pins for the oracle's row step: log-sum-exp and top-k with index tie-break."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import gto_oracle as orc


@pytest.mark.parametrize("V,scale", [(7, 1.0), (512, 2.5), (4096, 30.0)])
def test_lse_matches_naive_long_double(V, scale):
    rng = np.random.default_rng(V)
    z = rng.normal(size=V) * scale
    lse, ids, lp = orc.lse_and_topk(z, 3)
    naive = np.log(np.sum(np.exp(z.astype(np.longdouble))))
    assert abs(lse - float(naive)) < 1e-12 * max(1.0, abs(float(naive)))
    assert abs(lse - logsumexp(z)) < 1e-12 * max(1.0, abs(lse))
    # softmax sums to one, and the reported log-probabilities are its logs
    assert abs(np.sum(np.exp(z - lse)) - 1.0) < 1e-12
    assert np.allclose(np.exp(lp), softmax(z)[ids], rtol=1e-12)


def test_lse_shift_invariance_and_large_values():
    z = np.array([1000.0, 999.0, -1000.0])
    lse, _, _ = orc.lse_and_topk(z, 1)
    assert abs(lse - (1000.0 + np.log(1.0 + np.exp(-1.0)))) < 1e-12


def test_topk_is_full_sort_with_low_index_ties():
    rng = np.random.default_rng(1)
    for V in (5, 64, 1000):
        z = np.round(rng.normal(size=V) * 2.0) / 2.0       # many exact ties
        k = min(10, V)
        _, ids, lp = orc.lse_and_topk(z, k)
        brute = sorted(range(V), key=lambda i: (-z[i], i))[:k]
        assert list(ids) == brute
        assert np.all(np.diff(lp) <= 0)


def test_topk_constant_row_gives_first_ids():
    _, ids, lp = orc.lse_and_topk(np.zeros(33), 6)
    assert list(ids) == [0, 1, 2, 3, 4, 5]
    assert np.allclose(lp, -np.log(33.0))


def test_argmax_low_breaks_ties_to_lower_id():
    assert orc.argmax_low(np.array([1.0, 3.0, 3.0, 2.0])) == 1
