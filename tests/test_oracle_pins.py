"""Pins for the CPU oracle: it is checked against things other than itself.

Each test names the statement of the paper (or of plain linear algebra) it pins:
a hand-worked example, reductions to library routines, brute force over the
un-averaged objective (Eq. 4), closed forms and invariances.  None of these
tests needs a GPU.
"""
import os

import numpy as np
import pytest

from oracle import gq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
IMPLS = ["c", "numpy"]


def bf16_exact(rng, shape, scale=1.0):
    """Random values that are exactly representable in bf16, as (bits, fp64 values)."""
    bits = orc.f64_to_bf16_bits(rng.standard_normal(shape) * scale)
    return bits, orc.bf16_bits_to_f64(bits)


def read_fixture(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = [p.strip() for p in line.split("=", 1)]
        rows = [[float(t) for t in r.split()] for r in val.split(";")]
        out[key] = np.array(rows if len(rows) > 1 else rows[0], dtype=np.float64)
    return out


# --------------------------------------------------------------------------- P0
@pytest.mark.parametrize("impl", IMPLS)
def test_hand_example(impl):
    """Algorithm 1 (groups, saliency, guided Hessian) and Eq. 7 on the worked example in golden/hand_example.txt."""
    fx = read_fixture(os.path.join(GOLDEN, "hand_example.txt"))
    xb = orc.f64_to_bf16_bits(fx["X"])
    gb = orc.f64_to_bf16_bits(fx["grad"])
    W = fx["delta"].astype(np.float32)
    What = np.zeros_like(W)

    s2 = orc.saliency(gb, 2, impl=impl)
    np.testing.assert_array_equal(s2, fx["g2_s"])
    H2 = orc.hessian(xb, s2, impl=impl)
    np.testing.assert_array_equal(H2[0], fx["g2_H0"])
    np.testing.assert_array_equal(H2[1], fx["g2_H1"])
    np.testing.assert_array_equal(orc.objective(W, What, H2, impl=impl), fx["g2_loss"])
    assert fx["g2_loss"][-1] == fx["eq4_brute"]

    s1 = orc.saliency(gb, 1, impl=impl)
    np.testing.assert_array_equal(s1[0], fx["g1_s"])
    H1 = orc.hessian(xb, s1, impl=impl)
    np.testing.assert_array_equal(H1[0], fx["g1_H0"])
    np.testing.assert_array_equal(orc.objective(W, What, H1, impl=impl), fx["g1_loss"])
    # averaging: sum_k |J_k| H_k (g=2) == |J| H (g=1)
    np.testing.assert_array_equal(H2[0] + H2[1], 2 * H1[0])


# --------------------------------------------------------------------------- P1
@pytest.mark.parametrize("impl", IMPLS)
def test_unit_gradients_reduce_to_gram(impl):
    """g = 1 and dl/dZ == 1 give the unguided Hessian H = X^T X (Section 3.2)."""
    rng = np.random.default_rng(1)
    xb, x = bf16_exact(rng, (97, 24))
    gb = orc.f64_to_bf16_bits(np.ones((97, 16)))
    s = orc.saliency(gb, 1, impl=impl)
    np.testing.assert_array_equal(s, np.ones((1, 97)))
    H = orc.hessian(xb, s, impl=impl)
    ref = np.zeros((24, 24))
    for i in range(97):                       # textbook sum of outer products
        ref += np.outer(x[i], x[i])
    np.testing.assert_allclose(H[0], ref, rtol=1e-13, atol=1e-12)


# --------------------------------------------------------------------------- P2
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
def test_group_weighted_sum_is_group_independent(impl, g):
    """sum_k |J_k| H_k = X^T Diag(sum_j grad_ij^2) X for every g (definition of the group average)."""
    rng = np.random.default_rng(2)
    xb, x = bf16_exact(rng, (64, 12))
    gb, gr = bf16_exact(rng, (64, 32), 1e-2)
    H = orc.hessian(xb, orc.saliency(gb, g, impl=impl), impl=impl)
    m = 32 // g
    lhs = m * H.sum(axis=0)
    w = (gr * gr).sum(axis=1)
    rhs = np.einsum("i,ia,ib->ab", w, x, x)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12, atol=1e-18)


# --------------------------------------------------------------------------- P3
@pytest.mark.parametrize("impl", IMPLS)
def test_symmetric_psd(impl):
    rng = np.random.default_rng(3)
    xb, _ = bf16_exact(rng, (200, 20))
    gb, _ = bf16_exact(rng, (200, 8), 1e-3)
    H = orc.hessian(xb, orc.saliency(gb, 4, impl=impl), impl=impl)
    for k in range(4):
        np.testing.assert_allclose(H[k], H[k].T, rtol=1e-14, atol=0)
        ev = np.linalg.eigvalsh(0.5 * (H[k] + H[k].T))
        assert ev.min() >= -1e-10 * ev.max()
    if impl == "c":      # entry-by-entry loops are symmetric bit for bit
        for k in range(4):
            assert np.array_equal(H[k], H[k].T)


# --------------------------------------------------------------------------- P4
@pytest.mark.parametrize("impl", IMPLS)
def test_group_size_one_equals_unaveraged_objective(impl):
    """With one channel per group Eq. 7 is Eq. 4: sum_ij (dl/dZ_ij * x_i . (w_j - what_j))^2."""
    rng = np.random.default_rng(4)
    n, d_in, d_out = 9, 5, 6
    xb, x = bf16_exact(rng, (n, d_in))
    gb, gr = bf16_exact(rng, (n, d_out))
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    What = rng.standard_normal((d_out, d_in)).astype(np.float32)
    s = orc.saliency(gb, d_out, impl=impl)
    H = orc.hessian(xb, s, impl=impl)
    loss = orc.objective(W, What, H, impl=impl)
    brute = 0.0
    per_channel = [0.0] * d_out
    for i in range(n):
        for j in range(d_out):
            z = 0.0
            for a in range(d_in):
                z += float(x[i, a]) * (float(W[j, a]) - float(What[j, a]))
            t = (float(gr[i, j]) * z) ** 2
            brute += t
            per_channel[j] += t
    np.testing.assert_allclose(loss[:d_out], per_channel, rtol=1e-12)
    np.testing.assert_allclose(loss[d_out], brute, rtol=1e-12)


# --------------------------------------------------------------------------- P5
@pytest.mark.parametrize("impl", IMPLS)
def test_token_form_of_objective(impl):
    """loss_k = || Diag(sqrt(s_k)) X Delta_k ||_F^2, never forming H."""
    rng = np.random.default_rng(5)
    n, d_in, d_out, g = 50, 16, 12, 3
    xb, x = bf16_exact(rng, (n, d_in))
    gb, gr = bf16_exact(rng, (n, d_out), 1e-1)
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    What = (W + 0.01 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    s = orc.saliency(gb, g, impl=impl)
    loss = orc.objective(W, What, orc.hessian(xb, s, impl=impl), impl=impl)
    m = d_out // g
    delta = W.astype(np.float64) - What.astype(np.float64)
    for k in range(g):
        zk = x @ delta[k * m:(k + 1) * m].T                       # [n, m]
        sk = (gr[:, k * m:(k + 1) * m] ** 2).mean(axis=1)
        np.testing.assert_allclose(loss[k], (sk[:, None] * zk * zk).sum(), rtol=1e-12)
    np.testing.assert_allclose(loss[g], loss[:g].sum(), rtol=1e-15)


# --------------------------------------------------------------------------- P6
@pytest.mark.parametrize("impl", IMPLS)
def test_closed_forms(impl):
    rng = np.random.default_rng(6)
    n, d_in, g = 40, 7, 2
    gb, gr = bf16_exact(rng, (n, 4))
    s = orc.saliency(gb, g, impl=impl)
    # one-hot rows x_i = e_{a(i)}: H_k is diagonal with H_k[a,a] = sum_{i: a(i)=a} s_k[i]
    a_of = rng.integers(0, d_in, n)
    x = np.zeros((n, d_in))
    x[np.arange(n), a_of] = 1.0
    H = orc.hessian(orc.f64_to_bf16_bits(x), s, impl=impl)
    for k in range(g):
        diag = np.array([s[k][a_of == a].sum() for a in range(d_in)])
        np.testing.assert_allclose(H[k], np.diag(diag), rtol=1e-14, atol=0)
    # all rows equal x0 (distinct entries, so a transposed index would show): H_k = (sum_i s_k[i]) x0 x0^T
    x0 = np.array([1.0, -2.0, 3.0, 0.5, 0.0, 4.0, -1.5])
    xb = orc.f64_to_bf16_bits(np.tile(x0, (n, 1)))
    H = orc.hessian(xb, s, impl=impl)
    for k in range(g):
        np.testing.assert_allclose(H[k], s[k].sum() * np.outer(x0, x0), rtol=1e-13, atol=0)
    # a single token with a single non-zero gradient column lands in the right group only
    gsel = np.zeros((1, 8))
    gsel[0, 5] = 2.0
    s1 = orc.saliency(orc.f64_to_bf16_bits(gsel), 4, impl=impl)       # m = 2, channel 5 -> group 2
    np.testing.assert_array_equal(s1[:, 0], [0.0, 0.0, 2.0, 0.0])


# --------------------------------------------------------------------------- P7
@pytest.mark.parametrize("impl", IMPLS)
def test_scalings_permutations_and_chunking(impl):
    rng = np.random.default_rng(7)
    n, d_in, d_out, g = 75, 10, 8, 2
    xb, x = bf16_exact(rng, (n, d_in))
    gb, gr = bf16_exact(rng, (n, d_out))
    s = orc.saliency(gb, g, impl=impl)
    H = orc.hessian(xb, s, impl=impl)
    # grad -> 4 grad (exact in bf16): s, H scale by 16; grad_scale argument does the same
    s4 = orc.saliency(orc.f64_to_bf16_bits(4.0 * gr), g, impl=impl)
    np.testing.assert_allclose(s4, 16.0 * s, rtol=1e-15)
    np.testing.assert_allclose(orc.saliency(gb, g, grad_scale=4.0, impl=impl), 16.0 * s, rtol=1e-15)
    np.testing.assert_allclose(orc.saliency(gb, g, grad_scale=1e3, impl=impl), 1e6 * s, rtol=1e-14)
    # X -> 2 X: H scales by 4
    H2 = orc.hessian(orc.f64_to_bf16_bits(2.0 * x), s, impl=impl)
    np.testing.assert_allclose(H2, 4.0 * H, rtol=1e-15)
    # token permutation leaves H unchanged (up to summation order)
    p = rng.permutation(n)
    Hp = orc.hessian(xb[p], np.ascontiguousarray(s[:, p]), impl=impl)
    np.testing.assert_allclose(Hp, H, rtol=1e-12, atol=1e-15)
    # streaming over ragged chunks == one shot
    Hc = None
    for lo, hi in [(0, 1), (1, 33), (33, 33), (33, 75)]:
        Hc = orc.hessian(xb[lo:hi], np.ascontiguousarray(s[:, lo:hi]), H=Hc, impl=impl)
    np.testing.assert_allclose(Hc, H, rtol=1e-12, atol=1e-15)
    # permuting channels inside a group leaves s unchanged; across groups it does not
    m = d_out // g
    perm = np.concatenate([rng.permutation(m), m + rng.permutation(m)])
    np.testing.assert_allclose(orc.saliency(gb[:, perm], g, impl=impl), s, rtol=1e-14)
    swapped = np.concatenate([np.arange(m, 2 * m), np.arange(m)])
    np.testing.assert_allclose(orc.saliency(gb[:, swapped], g, impl=impl), s[::-1], rtol=1e-14)


# --------------------------------------------------------------------------- P8 / P9
@pytest.mark.parametrize("impl", IMPLS)
def test_diagonal_and_probe_forms_equal_the_full_hessian(impl):
    """hessian_diag and hessian_apply (the O(n d_in) checks used where the d_in x d_in oracle cannot go) against
    the full oracle matrix on small inputs, streamed in ragged chunks; and against what a planted mistake would
    give (unsquared x, s of the wrong group, a transposed probe product)."""
    rng = np.random.default_rng(21)
    n, d_in, g, nv = 131, 40, 3, 4
    xb, x = bf16_exact(rng, (n, d_in))
    s = rng.random((g, n)) * np.exp(rng.standard_normal(n))
    V = rng.standard_normal((nv, d_in))
    H = orc.hessian(xb, s, impl="c")
    diag, out = None, None
    for lo, hi in [(0, 50), (50, 51), (51, 51), (51, n)]:
        diag = orc.hessian_diag(xb[lo:hi], s[:, lo:hi], diag, impl=impl)
        out = orc.hessian_apply(xb[lo:hi], s[:, lo:hi], V, out, impl=impl)
    for k in range(g):
        np.testing.assert_allclose(diag[k], np.diag(H[k]), rtol=1e-12)
        np.testing.assert_allclose(out[k], (H[k] @ V.T).T, rtol=1e-11, atol=1e-11 * np.abs(out[k]).max())
    # planted mistakes are far outside those tolerances
    assert not np.allclose(diag[0], np.diag(H[1]), rtol=1e-3)
    assert not np.allclose(diag[0], (s[0][:, None] * np.abs(x)).sum(0), rtol=1e-3)
    assert not np.allclose(out[0, 0], H[0].T @ V[1], rtol=1e-3)
    # closed forms: one-hot rows give diag = per-feature sums of s and H v = diag * v
    hot = rng.integers(0, d_in, n)
    xh = np.zeros((n, d_in))
    xh[np.arange(n), hot] = 1.0
    xhb = orc.f64_to_bf16_bits(xh)
    d1 = orc.hessian_diag(xhb, s, impl=impl)
    o1 = orc.hessian_apply(xhb, s, V, impl=impl)
    for k in range(g):
        expect = np.bincount(hot, weights=s[k], minlength=d_in)
        np.testing.assert_allclose(d1[k], expect, rtol=1e-13)
        np.testing.assert_allclose(o1[k], expect[None, :] * V, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------- P10
@pytest.mark.parametrize("impl", IMPLS)
def test_objective_edge_cases(impl):
    rng = np.random.default_rng(10)
    n, d_in, d_out = 30, 6, 4
    xb, x = bf16_exact(rng, (n, d_in))
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    gb, _ = bf16_exact(rng, (n, d_out))
    H = orc.hessian(xb, orc.saliency(gb, 2, impl=impl), impl=impl)
    assert np.all(orc.objective(W, W.copy(), H, impl=impl) == 0.0)
    What = rng.standard_normal((d_out, d_in)).astype(np.float32)
    assert np.all(orc.objective(W, What, H, impl=impl) >= 0.0)
    # sign of delta is irrelevant
    np.testing.assert_allclose(orc.objective(W, What, H, impl=impl),
                               orc.objective(What, W, H, impl=impl), rtol=1e-14)
    # What = 0, g = 1, unit gradients: Eq. 1, || X W ||_F^2 with W = [w_1 ... w_dout]
    ones = orc.f64_to_bf16_bits(np.ones((n, d_out)))
    H1 = orc.hessian(xb, orc.saliency(ones, 1, impl=impl), impl=impl)
    loss = orc.objective(W, np.zeros_like(W), H1, impl=impl)
    np.testing.assert_allclose(loss[1], np.linalg.norm(x @ W.astype(np.float64).T, "fro") ** 2, rtol=1e-12)


# ------------------------------------------------------------- saliency from other dtypes and layouts
@pytest.mark.parametrize("impl", IMPLS)
def test_strided_typed_saliency(impl):
    """saliency_strided: the hand example in every dtype, equality with saliency() on bf16 rows, brute force in
    pure Python on a tiny strided fp16 / fp32 case (values widened exactly), a view with padded rows and a
    batch stride, half-precision subnormals and the gradient scale."""
    fx = read_fixture(os.path.join(GOLDEN, "hand_example.txt"))
    for dtype, arr in (("bf16", orc.f64_to_bf16_bits(fx["grad"])), ("fp16", fx["grad"].astype(np.float16)),
                       ("fp32", fx["grad"].astype(np.float32))):
        s2 = orc.saliency_strided(arr.reshape(1, 2, 2), dtype, 2, impl=impl)
        np.testing.assert_array_equal(s2, fx["g2_s"])
        s1 = orc.saliency_strided(arr.reshape(2, 1, 2), dtype, 1, impl=impl)
        np.testing.assert_array_equal(s1[0], fx["g1_s"])
    rng = np.random.default_rng(31)
    gb, _ = bf16_exact(rng, (24, 48), 1e-2)
    np.testing.assert_array_equal(orc.saliency_strided(gb.reshape(4, 6, 48), "bf16", 3, 2.0, impl=impl),
                                  orc.saliency(gb, 3, 2.0, impl="c"))
    for dtype, np_t in (("fp16", np.float16), ("fp32", np.float32)):
        wide = (rng.standard_normal((3, 5, 40)) * 1e-2).astype(np_t)          # [batch, seq, padded row]
        wide[0, 0, :4] = np.array([6e-8, -6e-8, 3e-5, 0.0]).astype(np_t)       # half subnormals (exact in fp32 too)
        view = wide[::2, :, :32]                          # rows padded from 32 to 40 elements, batch stride of two slabs
        got = orc.saliency_strided(view, dtype, 4, 3.0, impl=impl)
        assert got.shape == (4, 2 * 5)
        for b in range(2):
            for t in range(5):
                for k in range(4):
                    acc = 0.0
                    for j in range(8 * k, 8 * k + 8):
                        acc += (3.0 * float(view[b, t, j])) ** 2
                    assert abs(got[k, b * 5 + t] - acc / 8.0) <= 1e-15 * max(acc, 1e-300) + 1e-300
    with pytest.raises(ValueError):
        orc.saliency_strided(np.zeros((2, 2, 9), np.float32), "fp32", 2)
    with pytest.raises(ValueError):
        orc.saliency_strided(np.zeros((2, 2, 8), np.float32), "fp16", 2)


# ------------------------------------------------------------- C loops vs numpy
def test_c_loops_match_numpy_definitions():
    rng = np.random.default_rng(11)
    n, d_in, d_out, g = 300, 48, 64, 4
    xb, _ = bf16_exact(rng, (n, d_in))
    gb, _ = bf16_exact(rng, (n, d_out), 1e-3)
    W = (0.02 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    What = (W + 1e-3 * rng.standard_normal((d_out, d_in))).astype(np.float32)
    sc, sn = orc.saliency(gb, g, impl="c"), orc.saliency(gb, g, impl="numpy")
    np.testing.assert_allclose(sc, sn, rtol=1e-13)
    Hc, Hn = orc.hessian(xb, sc, impl="c"), orc.hessian(xb, sc, impl="numpy")
    np.testing.assert_allclose(Hc, Hn, rtol=1e-11, atol=1e-20)
    np.testing.assert_allclose(orc.objective(W, What, Hc, impl="c"),
                               orc.objective(W, What, Hc, impl="numpy"), rtol=1e-11)


def test_bad_shapes_are_rejected():
    gb = np.zeros((4, 6), dtype=np.uint16)
    with pytest.raises(ValueError):
        orc.saliency(gb, 4)            # 6 % 4 != 0
    with pytest.raises(ValueError):
        orc.hessian(np.zeros((4, 3), dtype=np.uint16), np.zeros((2, 5)))


def test_bf16_helpers_roundtrip():
    vals = np.array([0.0, 1.0, -2.5, 3.140625, 1e-3, 65280.0])
    bits = orc.f64_to_bf16_bits(vals)
    back = orc.bf16_bits_to_f64(bits)
    assert np.all(np.abs(back - vals) <= np.abs(vals) * 2.0 ** -8)
    np.testing.assert_array_equal(orc.f64_to_bf16_bits(back), bits)
    # ties to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.bf16_bits_to_f64(orc.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8])))[0] == 1.0
    assert orc.bf16_bits_to_f64(orc.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8])))[0] == 1.0 + 2.0 ** -6
