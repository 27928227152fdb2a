"""Pins for the LSE merge oracle (O2): split-and-merge equals unsplit attention at every split
point (Sec. 5.1: the partial outputs merge exactly), the algebra of the join, library routines."""
import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2609_14507_b200 import synth

MERGES = [pytest.param(c_oracle.merge, id="cpp"), pytest.param(np_oracle.merge, id="numpy")]


def _case(seed, N=48, Hq=8, Hkv=2, d=32):
    rng = np.random.default_rng(seed)
    return (synth.normal_bf16(rng, (Hq, d)), synth.normal_bf16(rng, (N, Hkv, d)),
            synth.normal_bf16(rng, (N, Hkv, d)))


@pytest.mark.parametrize("merge", MERGES)
def test_merge_at_every_split_point_equals_unsplit(merge):
    q, k, v = _case(11)
    N = k.shape[0]
    full = c_oracle.attend(q, k, v, np.arange(N), 0.21)
    for s in range(N + 1):
        a = c_oracle.attend(q, k, v, np.arange(0, s), 0.21)
        b = c_oracle.attend(q, k, v, np.arange(s, N), 0.21)
        O, lse = merge([a, b])
        np.testing.assert_allclose(O, full[0], rtol=1e-12, atol=1e-15, err_msg=f"split {s}")
        np.testing.assert_allclose(lse, full[1], rtol=1e-13, err_msg=f"split {s}")


@pytest.mark.parametrize("merge", MERGES)
def test_arbitrary_partitions_and_nway(merge):
    q, k, v = _case(12, N=61)
    N = k.shape[0]
    full = np_oracle.attend(q, k, v, np.arange(N), 0.3)
    rng = np.random.default_rng(0)
    for n_parts in (2, 3, 5, 9):
        label = rng.integers(0, n_parts, size=N)          # non-contiguous, some parts may be empty
        parts = [np_oracle.attend(q, k, v, np.nonzero(label == i)[0], 0.3) for i in range(n_parts)]
        O, lse = merge(parts)
        np.testing.assert_allclose(O, full[0], rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(lse, full[1], rtol=1e-13)


@pytest.mark.parametrize("merge", MERGES)
def test_associative_commutative_identity(merge):
    q, k, v = _case(13, N=30)
    a = c_oracle.attend(q, k, v, np.arange(0, 7), 0.2)
    b = c_oracle.attend(q, k, v, np.arange(7, 19), 0.2)
    c = c_oracle.attend(q, k, v, np.arange(19, 30), 0.2)
    left = merge([merge([a, b]), c])
    right = merge([a, merge([b, c])])
    flat = merge([c, a, b])
    for x in (right, flat):
        np.testing.assert_allclose(left[0], x[0], rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(left[1], x[1], rtol=1e-13)
    empty = (np.zeros_like(a[0]), np.full_like(a[1], -np.inf))
    same = merge([a, empty])
    np.testing.assert_allclose(same[0], a[0], rtol=1e-15)
    np.testing.assert_array_equal(same[1], a[1])
    both = merge([empty, empty])
    assert np.all(both[0] == 0) and np.all(np.isneginf(both[1]))


@pytest.mark.parametrize("merge", MERGES)
def test_lse_part_is_logaddexp_and_weights_are_softmax(merge):
    from scipy.special import logsumexp, softmax
    rng = np.random.default_rng(14)
    rows, dv, n = 6, 5, 4
    Os = rng.standard_normal((n, rows, dv))
    Ls = rng.standard_normal((n, rows)) * 10.0
    O, lse = merge([(Os[i], Ls[i]) for i in range(n)])
    np.testing.assert_allclose(lse, logsumexp(Ls, axis=0), rtol=1e-14)
    w = softmax(Ls, axis=0)
    np.testing.assert_allclose(O, np.einsum("nr,nrd->rd", w, Os), rtol=1e-13, atol=1e-15)
    # hand-derived: equal normalisers average the partial outputs, and LSE grows by ln 2
    O2, l2 = merge([(Os[0], Ls[0]), (Os[1], Ls[0])])
    np.testing.assert_allclose(O2, 0.5 * (Os[0] + Os[1]), rtol=1e-14)
    np.testing.assert_allclose(l2, Ls[0] + np.log(2.0), rtol=1e-14)


def test_two_way_form_matches_nway():
    rng = np.random.default_rng(15)
    Oa, Ob = rng.standard_normal((2, 7, 3))
    la, lb = rng.standard_normal((2, 7)) * 5
    lb[2] = -np.inf
    O2, l2 = np_oracle.merge2(Oa, la, Ob, lb)
    On, ln = c_oracle.merge([(Oa, la), (Ob, lb)])
    np.testing.assert_allclose(O2, On, rtol=1e-14)
    np.testing.assert_allclose(l2, ln, rtol=1e-14)
