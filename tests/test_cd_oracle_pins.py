"""Pins for the coordinate-descent oracle (oracle/cd_oracle.*): the three statements of cyclic CD agree, and
they agree with what the paper and the mathematics fix (hand example, closed forms, descent)."""
import os

import numpy as np
import pytest

from oracle import cd_oracle as cdo
from oracle import gq_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def make_problem(seed, d_in, d_out, g, m, n=80):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d_in)) * np.exp(0.5 * rng.standard_normal(d_in))
    H = np.stack([(X * rng.random((n, 1))).T @ X for _ in range(g)]).astype(np.float32)
    W = (0.1 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    cb = np.sort(0.12 * rng.standard_normal((d_out, m)), axis=1).astype(np.float32)
    W0, _ = cdo.round_to_codebook(W, cb)
    return W, W0.astype(np.float32), cb, H


def test_hand_example():
    H = np.array([[[2.0, 1.0], [1.0, 2.0]]], dtype=np.float32)
    cb = np.array([[0.0, 1.0]], dtype=np.float32)
    for line in open(os.path.join(HERE, "golden", "cd_hand_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, rest = line.split(None, 1)
        w, start, after, _targets = [np.array(p.split(), dtype=np.float64) for p in rest.split("|")]
        for fn in (lambda *a: cdo.cd(*a, 1, 128), lambda *a: cdo.cd_rowwise(*a, 1), lambda *a: cdo.cd_naive(*a, 1)):
            What, Q = fn(w[None].astype(np.float32), start[None].astype(np.float32), cb, H)
            assert np.array_equal(What[0], after.astype(np.float32)), name
            assert np.array_equal(Q[0], after.astype(np.int32)), name


@pytest.mark.parametrize("seed,d_in,d_out,g,m,b", [(0, 24, 8, 2, 4, 8), (1, 37, 6, 3, 8, 16), (2, 16, 4, 1, 2, 5),
                                                   (3, 50, 4, 2, 16, 128)])
def test_three_statements_agree(seed, d_in, d_out, g, m, b):
    """Algorithm 4 (any block size, ragged last block), Algorithm 3 and exhaustive-evaluation CD take the same
    decisions: the closed form of Eq. 10 is the exact coordinate minimiser and deferring corrections changes
    nothing."""
    W, W0, cb, H = make_problem(seed, d_in, d_out, g, m)
    ref = cdo.cd_naive(W, W0, cb, H, 2)
    for got in (cdo.cd(W, W0, cb, H, 2, b), cdo.cd(W, W0, cb, H, 2, 10 ** 6), cdo.cd(W, W0, cb, H, 2, 1),
                cdo.cd_rowwise(W, W0, cb, H, 2)):
        assert np.array_equal(got[1], ref[1])
        assert np.array_equal(got[0], ref[0])


def test_descent_and_fixed_point():
    """CD started from a feasible point never increases any channel's objective (Proposition 1, second
    inequality), and a point it no longer changes is a fixed point of further cycles."""
    W, W0, cb, H = make_problem(5, 40, 12, 2, 4)
    mk = W.shape[0] // H.shape[0]

    def per_channel(What):
        return np.array([cdo.channel_objective(What[j].astype(np.float64) - W[j], H[j // mk].astype(np.float64))
                         for j in range(W.shape[0])])

    prev, cur = W0, per_channel(W0)
    for _ in range(6):
        nxt, _ = cdo.cd(W, prev, cb, H, 1, 8)
        f = per_channel(nxt)
        assert np.all(f <= cur * (1 + 1e-12) + 1e-300)
        prev, cur = nxt, f
    # the group totals are what the objective of Eq. 7 reports
    tot = orc.objective(W, prev, H.astype(np.float64))
    assert np.allclose(tot[:-1], cur.reshape(H.shape[0], mk).sum(1), rtol=1e-10)
    again, _ = cdo.cd(W, prev, cb, H, 3, 8)
    stable, _ = cdo.cd(W, again, cb, H, 1, 8)
    assert np.all(per_channel(stable) <= per_channel(again) * (1 + 1e-12))


def test_diagonal_hessian_is_plain_rounding():
    """With a diagonal H the coordinates decouple: one cycle gives nearest-value rounding of W."""
    rng = np.random.default_rng(7)
    d_in, d_out, m = 30, 5, 4
    H = np.diag(rng.random(d_in) + 0.1)[None].astype(np.float32)
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    cb = np.sort(rng.standard_normal((d_out, m)), axis=1).astype(np.float32)
    start = np.repeat(cb[:, :1], d_in, axis=1)
    What, Q = cdo.cd(W, start, cb, H, 1, 7)
    val, q = cdo.round_to_codebook(W, cb)
    assert np.array_equal(Q, q) and np.array_equal(What, val.astype(np.float32))


def test_ties_and_dead_features():
    cb = np.array([[0.0, 1.0, 2.0]], dtype=np.float32)
    H = np.array([[[1.0, 0.0, 0.0], [0.0, 0.0, 0.0], [0.0, 0.0, 4.0]]], dtype=np.float32)   # feature 1 never fired
    W = np.array([[0.5, 1.5, 1.49]], dtype=np.float32)
    What, Q = cdo.cd(W, np.zeros((1, 3), np.float32), cb, H, 1, 128)
    assert Q.tolist() == [[0, 1, 1]]          # exact ties go to the smaller index; dead feature: nearest to W
    assert What.tolist() == [[0.0, 1.0, 1.0]]
