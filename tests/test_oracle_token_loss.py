"""Pins for the token-level loss (Eq. 13, App. B): library cross-entropy with soft targets and
its autograd derivative, the identity H(p, q) = KL(p || q) + H(p) with scipy's entropies, and
the special cases that follow from the definition."""
import numpy as np
import pytest
import torch
from scipy.special import softmax
from scipy.stats import entropy

from oracle import gto_oracle as orc


@pytest.mark.parametrize("seed", range(3))
def test_matches_torch_soft_target_cross_entropy_and_autograd(seed):
    rng = np.random.default_rng(seed)
    V = 37
    zd, zt = rng.normal(size=V) * 3, rng.normal(size=V) * 3
    H, grad = orc.token_loss(zd, zt)
    z = torch.tensor(zd, dtype=torch.float64, requires_grad=True)
    target = torch.softmax(torch.tensor(zt, dtype=torch.float64), dim=0)
    loss = torch.nn.functional.cross_entropy(z[None, :], target[None, :])
    loss.backward()
    assert H == pytest.approx(float(loss), rel=1e-12)
    assert np.allclose(grad, z.grad.numpy(), atol=1e-13)
    assert abs(grad.sum()) < 1e-12


def test_cross_entropy_is_kl_plus_target_entropy():
    rng = np.random.default_rng(5)
    zd, zt = rng.normal(size=50) * 2, rng.normal(size=50) * 2
    H, _ = orc.token_loss(zd, zt)
    p, q = softmax(zt), softmax(zd)
    assert H == pytest.approx(entropy(p, q) + entropy(p), rel=1e-12)


def test_identical_distributions_and_shift_invariance():
    rng = np.random.default_rng(6)
    z = rng.normal(size=20)
    H, grad = orc.token_loss(z, z + 3.5)           # softmax ignores a constant shift
    assert H == pytest.approx(entropy(softmax(z)), rel=1e-12)
    assert np.allclose(grad, 0.0, atol=1e-14)


def test_one_hot_target_gives_the_negative_log_likelihood():
    z = np.array([0.3, -1.2, 2.0, 0.1])
    zt = np.array([0.0, 0.0, 800.0, 0.0])           # target puts all mass on token 2
    H, grad = orc.token_loss(z, zt)
    lp = z - np.log(np.sum(np.exp(z)))
    assert H == pytest.approx(-lp[2], rel=1e-12)
    want = np.exp(lp)
    want[2] -= 1.0
    assert np.allclose(grad, want, atol=1e-13)


def test_reduced_vocabulary_renormalises_the_target_over_the_mapped_ids():
    rng = np.random.default_rng(7)
    Vt, Vd = 40, 9
    d2t = np.sort(rng.choice(Vt, size=Vd, replace=False))
    zd, zt = rng.normal(size=Vd), rng.normal(size=Vt) * 2
    H, grad = orc.token_loss(zd, zt, d2t)
    H2, grad2 = orc.token_loss(zd, zt[d2t])
    assert H == H2 and np.array_equal(grad, grad2)
    # a transposed operand (draft as teacher) gives a different value
    assert abs(orc.token_loss(zt[d2t], zd)[0] - H) > 1e-3
