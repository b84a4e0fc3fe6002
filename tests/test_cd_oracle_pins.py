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
        w, start, after, targets = [np.array(p.split(), dtype=np.float64) for p in rest.split("|")]
        for fn in (lambda *a: cdo.cd(*a, 1, 128), lambda *a: cdo.cd_rowwise(*a, 1), lambda *a: cdo.cd_naive(*a, 1)):
            What, Q = fn(w[None].astype(np.float32), start[None].astype(np.float32), cb, H)
            assert np.array_equal(What[0], after.astype(np.float32)), name
            assert np.array_equal(Q[0], after.astype(np.int32)), name
        # the arguments of Round_j written out by hand in the file: coordinate 1 sees the starting point,
        # coordinate 2 sees coordinate 1 already updated
        cur = start.copy()
        for i in range(2):
            t, mag = cdo.coordinate_target(w, cur, H[0], i)
            assert abs(t - targets[i]) <= 1e-12, (name, i, t)
            assert abs(mag - (abs(w[i]) + 0.5 * abs(cur[1 - i] - w[1 - i]))) <= 1e-12, (name, i, mag)
            cur[i] = after[i]


def test_coordinate_target_is_the_minimiser_of_the_one_coordinate_quadratic():
    """Eq. 10 before rounding: with every other coordinate of the channel held fixed, the channel objective as a
    function of the value t of coordinate i is a parabola; its vertex, found here from three evaluations of the
    objective alone (no algebra on H), is what coordinate_target must return.  The second return value is the
    sum of the magnitudes of the terms, re-added here one by one."""
    rng = np.random.default_rng(11)
    for trial in range(20):
        d = int(rng.integers(2, 9))
        A = rng.standard_normal((d + 3, d))
        Hk = A.T @ A
        w = rng.standard_normal(d)
        what = rng.standard_normal(d)
        i = int(rng.integers(0, d))

        def f(t):
            trial_w = what.copy()
            trial_w[i] = t
            return cdo.channel_objective(trial_w - w, Hk)

        fm, f0, fp = f(-1.0), f(0.0), f(1.0)
        vertex = 0.5 * (fm - fp) / (fm - 2.0 * f0 + fp)
        t, mag = cdo.coordinate_target(w, what, Hk, i)
        assert abs(t - vertex) <= 1e-9 * max(1.0, abs(vertex)), (trial, t, vertex)
        assert f(t) <= min(f(t + 1e-3), f(t - 1e-3))
        expect_mag = abs(w[i])
        for c in range(d):
            if c != i:
                expect_mag += abs(Hk[i, c] / Hk[i, i] * (what[c] - w[c]))
        assert abs(mag - expect_mag) <= 1e-12 * expect_mag
    # a feature that never fired: the target is the weight itself
    Hk = np.diag([1.0, 0.0, 2.0])
    t, mag = cdo.coordinate_target(np.array([0.3, -0.7, 0.1]), np.array([1.0, 1.0, 1.0]), Hk, 1)
    assert t == -0.7 and mag == 0.7


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


# ------------------------------------------------------------------------------------------ codebook step
def test_codebook_step_is_the_least_squares_solution():
    """Eq. 8 against the formulation the paper gives to its solver: min_c || L^T (P c - w) ||_2 with
    H = L L^T (library least squares), against the diagonal closed form, and against perturbations."""
    from scipy.linalg import cholesky, lstsq
    W, W0, cb, H = make_problem(9, 40, 6, 2, 4, n=200)
    _, Q = cdo.round_to_codebook(W, cb)
    C = cdo.codebook_update(W, Q, H, 4, lam=0.0)
    mk = 3
    for j in range(6):
        Hk = H[j // mk].astype(np.float64)
        L = cholesky(Hk, lower=True)
        P = cdo.one_hot(Q[j], 4)
        ref, *_ = lstsq(L.T @ P, L.T @ W[j].astype(np.float64))
        assert np.allclose(C[j], ref, rtol=1e-7, atol=1e-10)
        f_opt = cdo.channel_objective(P @ C[j] - W[j], Hk)
        rng = np.random.default_rng(j)
        for _ in range(5):                                   # no perturbed codebook does better
            f = cdo.channel_objective(P @ (C[j] + 1e-3 * rng.standard_normal(4)) - W[j], Hk)
            assert f >= f_opt
        assert f_opt <= cdo.channel_objective(P @ cb[j].astype(np.float64) - W[j], Hk) * (1 + 1e-12)
    # diagonal H: every level becomes the H_ii-weighted mean of the weights assigned to it
    h = np.random.default_rng(1).random(40) + 0.1
    Cd = cdo.codebook_update(W, Q, np.stack([np.diag(h)] * 2), 4, lam=0.0)
    for j in range(6):
        for q in range(4):
            sel = Q[j] == q
            if sel.any():
                assert np.isclose(Cd[j, q], (h[sel] * W[j, sel]).sum() / h[sel].sum(), rtol=1e-10)
    # a level nobody uses: lam keeps the system solvable and gives that level the value 0
    Q1 = Q.copy()
    Q1[Q1 == 3] = 2
    C1 = cdo.codebook_update(W, Q1, H, 4, lam=1e-7)
    assert np.all(C1[:, 3] == 0.0) and np.all(np.isfinite(C1))


def test_lnq_descends():
    """Proposition 1: the objective of every channel is non-increasing over the LNQ iterations."""
    W, W0, cb, H = make_problem(10, 48, 8, 2, 4, n=200)
    _, Q0 = cdo.round_to_codebook(W, cb)
    mk = 4

    def per_channel(What):
        return np.array([cdo.channel_objective(What[j].astype(np.float64) - W[j], H[j // mk].astype(np.float64))
                         for j in range(8)])

    f_prev = per_channel(W0)
    Q = Q0
    for t in range(3):
        c = cdo.codebook_update(W, Q, H, 4).astype(np.float32)
        f_c = per_channel(np.take_along_axis(c, Q, axis=1))
        assert np.all(f_c <= f_prev * (1 + 1e-5))            # codebook step (fp32 codebook: 1e-5 slack)
        What, Q = cdo.cd(W, np.take_along_axis(c, Q, axis=1), c, H, 2, 16)
        f_prev = per_channel(What)
        assert np.all(f_prev <= f_c * (1 + 1e-12))           # CD
    What, Qf, cf = cdo.lnq(W, Q0, H, 4, T=3, K=2, b=16)
    assert np.all(per_channel(What) <= f_prev * (1 + 1e-5))


def test_lnq_is_algorithm_2_in_order():
    """Algorithm 2: T times (codebook step, then K CD cycles), then one more codebook step.  lnq() must equal that
    sequence composed here by hand from codebook_update and cd, bit for bit, and every deviation from the order
    (no final codebook step, CD before the codebook step, one round fewer) must give another result on this
    problem."""
    W, W0, cb, H = make_problem(12, 40, 8, 2, 4, n=160)
    _, Q0 = cdo.round_to_codebook(W, cb)
    m, T, K, b = 4, 2, 2, 16

    def cstep(Q):
        c = cdo.codebook_update(W, Q, H, m).astype(np.float32)
        return c, np.take_along_axis(c, Q, axis=1)

    Q = Q0.copy()
    for _ in range(T):
        c, What = cstep(Q)
        What, Q = cdo.cd(W, What, c, H, K, b)
    Q_before_final, What_before_final, c_before_final = Q, What, c
    c, What = cstep(Q)
    got = cdo.lnq(W, Q0, H, m, T=T, K=K, b=b)
    assert np.array_equal(got[1], Q) and np.array_equal(got[0], What) and np.array_equal(got[2], c)
    # without the final codebook step the codebook (and W_hat) would be the previous round's
    assert not np.array_equal(got[2], c_before_final)
    assert not np.array_equal(got[0], What_before_final)
    # the final step can only lower every channel's objective, and lowers some
    mk = W.shape[0] // H.shape[0]
    f = lambda Wh: np.array([cdo.channel_objective(Wh[j].astype(np.float64) - W[j], H[j // mk].astype(np.float64))
                             for j in range(W.shape[0])])
    assert np.all(f(got[0]) <= f(What_before_final) * (1 + 1e-5)) and np.any(f(got[0]) < f(What_before_final))
    # CD first, codebook step second (the wrong order) ends elsewhere
    Qw, cw = Q0.copy(), cb.copy()
    Whw = np.take_along_axis(cw, Qw, axis=1)
    for _ in range(T):
        Whw, Qw = cdo.cd(W, Whw, cw, H, K, b)
        cw, Whw = cstep(Qw)
    assert not (np.array_equal(Qw, got[1]) and np.array_equal(cw, got[2]))
    # T - 1 rounds end elsewhere, T = 0 is the codebook step alone
    fewer = cdo.lnq(W, Q0, H, m, T=T - 1, K=K, b=b)
    assert not np.array_equal(fewer[2], got[2])
    only = cdo.lnq(W, Q0, H, m, T=0, K=K, b=b)
    c0, What0 = cstep(Q0)
    assert np.array_equal(only[1], Q0) and np.array_equal(only[2], c0) and np.array_equal(only[0], What0)
