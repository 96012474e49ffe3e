"""Pins for debiasing / standardisation (Eq. 9-10) and the clipped surrogate (Eq. 11-12)."""
import numpy as np
import pytest
import torch
from scipy.stats import zscore

from oracle import gto_oracle as orc


def test_advantages_match_scipy_zscore_and_sum_to_zero():
    rng = np.random.default_rng(0)
    B, m = 32, 8
    rc, rr = rng.normal(size=B) + 3, rng.normal(size=B) + 3
    R, A = orc.group_advantages(rc, rr, m, delta=0.0)
    assert np.allclose(R, rc - rr)
    for k0 in range(0, B, m):
        assert np.allclose(A[k0:k0 + m], zscore(R[k0:k0 + m], ddof=0), atol=1e-12)
        assert abs(A[k0:k0 + m].sum()) < 1e-12
    R, A = orc.group_advantages(rc, rr, m, delta=1e-6)
    for k0 in range(0, B, m):
        grp = R[k0:k0 + m]
        sd = grp.std()
        assert abs(A[k0:k0 + m].sum()) < 1e-9
        assert np.sum(A[k0:k0 + m] ** 2) == pytest.approx(m * (sd / (sd + 1e-6)) ** 2, rel=1e-12)
    _, Au = orc.group_advantages(rc, rr, m, delta=0.0, unbiased=True)
    assert np.allclose(Au[:m], zscore(R[:m], ddof=1), atol=1e-12)


def test_advantages_special_cases():
    rc = np.array([1.0, 2.0, 4.0, 8.0])
    _, A1 = orc.group_advantages(rc, np.zeros(4), 1)
    assert np.all(A1 == 0.0)                                    # m = 1
    _, A0 = orc.group_advantages(rc, rc, 4)
    assert np.all(A0 == 0.0)                                    # identical trees
    _, A = orc.group_advantages(rc, np.zeros(4), 4, delta=0.0)
    _, A2 = orc.group_advantages(3 * rc + 7, np.zeros(4), 4, delta=0.0)
    assert np.allclose(A, A2)                                   # affine invariance
    _, An = orc.group_advantages(rc, np.ones(4), 4, delta=0.0, debias=False)
    assert np.allclose(An, A)


# factor on the summed group losses for each seed of the autograd pin: 1, and the
# omega / K = 0.5 / 16 a trainer passes with the settings of App. B
GRAD_SCALES = [1.0, 0.5 / 16, 3.0, 0.5 / 16]


def torch_loss(z, rows_tok, old, adv, m, eps):
    """Eq. 11-12 written with torch ops on leaf logits z[b][j]; autograd differentiates."""
    total = 0.0
    for b, (zs, toks) in enumerate(zip(z, rows_tok)):
        l = len(toks)
        lp = sum(torch.log_softmax(zs[j], dim=0)[toks[j]] for j in range(l)) if l else torch.tensor(0.0, dtype=torch.float64)
        s = torch.exp((lp - sum(old[b][:l])) / max(l, 1))
        a = torch.tensor(adv[b], dtype=torch.float64)
        total = total + (-1.0 / m) * torch.minimum(s * a, torch.clamp(s, 1 - eps, 1 + eps) * a)
    return total


@pytest.mark.parametrize("seed", range(4))
def test_gradient_matches_autograd_and_finite_differences(seed):
    rng = np.random.default_rng(seed)
    B, m, D, V, eps = 16, 4, 3, 6, 0.2
    lens = rng.integers(0, D + 1, size=B)
    rows = [[rng.normal(size=V) for _ in range(l)] for l in lens]
    toks = [[int(rng.integers(0, V)) for _ in range(l)] for l in lens]
    adv = rng.normal(size=B)
    path_logp = np.zeros((B, D))
    lse = [[np.log(np.sum(np.exp(r))) for r in rs] for rs in rows]
    for b in range(B):
        for j in range(lens[b]):
            path_logp[b, j] = rows[b][j][toks[b][j]] - lse[b][j]
    old = path_logp + rng.normal(size=(B, D)) * 0.6       # some ratios leave the clip range
    scale = GRAD_SCALES[seed]
    sur = orc.clipped_surrogate(path_logp, old, lens, adv, m, eps=eps, grad_scale=scale)
    assert (~sur["active"]).any() and sur["active"].any()
    z = [[torch.tensor(r, dtype=torch.float64, requires_grad=True) for r in rs] for rs in rows]
    loss = torch_loss(z, toks, old, adv, m, eps)
    assert float(loss.detach()) == pytest.approx(float(sur["loss"].sum()), rel=1e-12)
    (scale * loss).backward()           # the gradient is that of grad_scale * sum_k loss_k
    for b in range(B):
        got = orc.surrogate_grad_rows(rows[b], lse[b], toks[b], sur["coeff"][b], D, V)
        for j in range(D):
            if j < lens[b]:
                want = z[b][j].grad.numpy() if z[b][j].grad is not None else np.zeros(V)
                assert np.allclose(got[j], want, atol=1e-12)
                assert abs(got[j].sum()) < 1e-12           # onehot - softmax sums to zero
            else:
                assert np.all(got[j] == 0.0)
        if not sur["active"][b]:
            assert np.all(got == 0.0)
    # central finite differences on one active position
    b = int(np.flatnonzero(sur["active"] & (lens > 0))[0])
    h = 1e-6
    for j in range(lens[b]):
        for v in range(V):
            def total(delta):
                rr = [r.copy() for r in rows[b]]
                rr[j][v] += delta
                pl = path_logp.copy()
                for jj in range(lens[b]):
                    pl[b, jj] = rr[jj][toks[b][jj]] - np.log(np.sum(np.exp(rr[jj])))
                return scale * orc.clipped_surrogate(pl, old, lens, adv, m, eps=eps)["loss"].sum()
            fd = (total(h) - total(-h)) / (2 * h)
            got = orc.surrogate_grad_rows(rows[b], lse[b], toks[b], sur["coeff"][b], D, V)[j, v]
            assert abs(fd - got) < 1e-7


def test_ratio_is_one_when_old_equals_current_and_clip_edges():
    pl = np.array([[-1.0, -2.0], [-0.5, 0.0]])
    sur = orc.clipped_surrogate(pl, pl, [2, 1], [1.0, -1.0], 2)
    assert np.all(sur["ratio"] == 1.0) and sur["active"].all()
    assert sur["loss"][0] == pytest.approx(0.0)
    assert sur["coeff"][0] == pytest.approx(-0.5 * 1.0 * 1.0 / 2)
    # length 0: ratio 1, nothing to differentiate through
    sur = orc.clipped_surrogate(pl, pl - 1.0, [0, 0], [1.0, -1.0], 2)
    assert np.all(sur["ratio"] == 1.0)
    # geometric mean: (sum diff) / l
    old = pl.copy(); old[0] -= np.log(1.1)
    sur = orc.clipped_surrogate(pl, old, [2, 1], [1.0, -1.0], 2)
    assert sur["ratio"][0] == pytest.approx(1.1)
    # clipped cases: A > 0 with s > 1+eps, A < 0 with s < 1-eps
    old = pl.copy(); old[0] -= np.log(1.5); old[1, 0] += np.log(2.0)
    sur = orc.clipped_surrogate(pl, old, [2, 1], [1.0, -1.0], 2, eps=0.2)
    assert sur["ratio"][0] == pytest.approx(1.5) and sur["ratio"][1] == pytest.approx(0.5)
    assert not sur["active"].any() and np.all(sur["coeff"] == 0.0)
    assert sur["loss"][0] == pytest.approx(-0.5 * (1.2 * 1.0 + 0.8 * -1.0))
    # not clipped in the pessimistic direction: A > 0 with s < 1-eps stays active
    sur = orc.clipped_surrogate(pl, old, [2, 1], [-1.0, 1.0], 2, eps=0.2)
    assert sur["active"].all()


def test_sample_groups_respects_the_constraints_and_reaches_every_placement():
    """Eq. 6-7: 1 <= t_k <= s - m + 1, t_{k+1} >= t_k + m.  Brute force on a tiny case: when
    the uniforms sweep a fine grid every admissible placement is produced, each as often as
    its offsets have orderings (the law of K independent sorted offsets: valid, not uniform)."""
    import itertools
    s, m, K = 9, 2, 3
    placements = [t for t in itertools.combinations(range(1, s - m + 2), K)
                  if all(t[i + 1] >= t[i] + m for i in range(K - 1))]
    counts = {t: 0 for t in placements}
    n = s - K * m + 1
    grid = [(i + 0.5) / n for i in range(n)]
    for u in itertools.product(grid, repeat=K):
        t = tuple(orc.sample_groups(s, m, K, u))
        assert t in counts
        counts[t] += 1
    # sorted K-multisets of n gap values: each placement corresponds to one multiset; the
    # number of orderings differs between multisets, so compare with the multinomial count
    from math import factorial
    from collections import Counter
    for t, c in counts.items():
        gaps = [t[i] - 1 - i * m for i in range(K)]
        perms = factorial(K)
        for rep in Counter(gaps).values():
            perms //= factorial(rep)
        assert c == perms
    assert orc.sample_groups(16, 8, 2, [0.3, 0.9]) == [1, 9]       # no slack: the partition
    assert orc.sample_groups(10, 4, 0, []) == []
    rng = np.random.default_rng(0)
    for _ in range(200):
        s_, m_ = int(rng.integers(8, 300)), int(rng.integers(1, 9))
        K_ = int(rng.integers(0, s_ // m_ + 1))
        t = orc.sample_groups(s_, m_, K_, rng.random(K_))
        assert all(1 <= x <= s_ - m_ + 1 for x in t)
        assert all(t[i + 1] >= t[i] + m_ for i in range(len(t) - 1))
