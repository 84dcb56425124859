"""Pins for the CPU oracle: every oracle function is checked against something other than
itself -- values the paper fixes (Eq. 3), brute force with a library matmul, closed forms,
exact rational arithmetic and invariants.  No GPU needed."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import bnn_oracle as o
from paper_1706_09453_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def np_pack(bits):
    """Independent packer: numpy packbits, LSB first, viewed as little-endian uint32."""
    m, k = bits.shape
    kw = (k + 31) // 32
    pad = np.zeros((m, kw * 32), dtype=np.uint8)
    pad[:, :k] = bits
    return np.packbits(pad, axis=1, bitorder="little").view("<u4").reshape(m, kw)


def pm1(bits):
    return bits.astype(np.float64) * 2.0 - 1.0


# ---------------------------------------------------------------- Sign / pack (Eq. 3)
def test_sign_matches_eq3_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "sign_eq3.txt")) if not l.startswith("#")]
    assert len(rows) == 11
    for x, eq3, zpos in rows:
        assert o.sign(float(x), o.SIGN_ZERO_NEG) == int(eq3), x
        assert o.sign(float(x), o.SIGN_ZERO_POS) == int(zpos), x


@pytest.mark.parametrize("mode", [o.SIGN_ZERO_POS, o.SIGN_ZERO_NEG])
@pytest.mark.parametrize("k", [1, 31, 32, 33, 100])
def test_sign_pack_against_numpy_packbits(mode, k):
    rng = np.random.default_rng(k)
    x = rng.standard_normal((7, k)).astype(np.float32)
    x[rng.random((7, k)) < 0.2] = 0.0
    x[0, 0] = -0.0
    x[1, 0] = np.nan
    x[2, 0] = np.float32(1e-45)   # denormal
    x[3, 0] = -np.float32(1e-45)
    with np.errstate(invalid="ignore"):
        bits = (x > 0) if mode == o.SIGN_ZERO_NEG else (x >= 0)
    got = o.sign_pack(x, mode)
    assert got.dtype == np.uint32 and got.shape == (7, (k + 31) // 32)
    np.testing.assert_array_equal(got, np_pack(bits.astype(np.uint8)))
    # unpack(pack(x)) == Sign(x), and the pad bits of the last word are zero
    np.testing.assert_array_equal(o.unpack_pm1(got, k), np.where(bits, 1, -1))
    if k % 32:
        assert (got[:, -1] >> np.uint32(k % 32)).max() == 0


def test_sign_pack_pitch_words_are_zeroed():
    x = np.ones((3, 40), dtype=np.float32)
    got = o.sign_pack(x, pitch=4)
    assert got.shape == (3, 4)
    np.testing.assert_array_equal(got[:, 2:], 0)
    np.testing.assert_array_equal(got[:, 0], 0xFFFFFFFF)
    np.testing.assert_array_equal(got[:, 1], 0xFF)


# ---------------------------------------------------------------- +-1 x +-1 dot products
@pytest.mark.parametrize("k", [1, 31, 32, 33, 127, 440, 600])
def test_xnor_gemm_brute_force_float_matmul(k):
    a = wl.make_bit_matrix(5, k, 0.5, [10, k])
    w = wl.make_bit_matrix(9, k, 0.5, [11, k])
    d = o.xnor_gemm(np_pack(a), np_pack(w), k)
    ref = pm1(a) @ pm1(w).T   # exact in float64
    assert d.dtype == np.int32 and d.shape == (5, 9)
    np.testing.assert_array_equal(d, ref.astype(np.int64))


def test_xnor_gemm_invariants():
    k = 200
    a = wl.make_bit_matrix(6, k, 0.5, 1)
    w = wl.make_bit_matrix(4, k, 0.3, 2)
    ap, wp = np_pack(a), np_pack(w)
    d = o.xnor_gemm(ap, wp, k)
    assert np.abs(d).max() <= k
    assert np.all((d - k) % 2 == 0)
    # dot(a, a) = K, dot(a, not a) = -K
    np.testing.assert_array_equal(np.diag(o.xnor_gemm(ap, ap, k)), k)
    np.testing.assert_array_equal(np.diag(o.xnor_gemm(ap, np_pack(1 - a), k)), -k)
    # flipping the sign of one weight row negates that output column only
    w2 = w.copy()
    w2[2] = 1 - w2[2]
    d2 = o.xnor_gemm(ap, np_pack(w2), k)
    np.testing.assert_array_equal(d2[:, 2], -d[:, 2])
    np.testing.assert_array_equal(np.delete(d2, 2, 1), np.delete(d, 2, 1))
    # a common permutation of k changes nothing
    perm = np.random.default_rng(3).permutation(k)
    np.testing.assert_array_equal(o.xnor_gemm(np_pack(a[:, perm]), np_pack(w[:, perm]), k), d)
    # XNOR identity  dot = K - 2 popc(a xor w)  and AND identity
    # dot = K - 2 popc(a) - 2 popc(w) + 4 popc(a and w)   (checked with numpy on the bits)
    x = (a[:, None, :] ^ w[None, :, :]).sum(-1).astype(np.int64)
    np.testing.assert_array_equal(d, k - 2 * x)
    an = (a[:, None, :] & w[None, :, :]).sum(-1).astype(np.int64)
    np.testing.assert_array_equal(
        d, k - 2 * a.sum(1, dtype=np.int64)[:, None] - 2 * w.sum(1, dtype=np.int64)[None, :] + 4 * an)


def test_xnor_gemm_ignores_pad_bits_and_pitch():
    k = 45
    a = wl.make_bit_matrix(3, k, 0.5, 5)
    w = wl.make_bit_matrix(4, k, 0.5, 6)
    ap = np.zeros((3, 4), np.uint32)
    wp = np.zeros((4, 8), np.uint32)
    ap[:, :2] = np_pack(a)
    wp[:, :2] = np_pack(w)
    np.testing.assert_array_equal(o.xnor_gemm(ap, wp, k), (pm1(a) @ pm1(w).T).astype(np.int64))


@pytest.mark.parametrize("p", [0.5, 0.1])
def test_xnor_gemm_moments_closed_form(p):
    """iid Bernoulli(p) bits: E[dot] = K(2q-1), Var[dot] = K(1-(2q-1)^2), q = p^2+(1-p)^2."""
    m, n, k = 64, 64, 1024
    ap = wl.make_bit_planes(m, k, p, [7, int(p * 10)])
    wp = wl.make_bit_planes(n, k, p, [8, int(p * 10)])
    d = o.xnor_gemm(ap, wp, k).astype(np.float64)
    q = p * p + (1 - p) * (1 - p)
    mean, var = k * (2 * q - 1), k * (1 - (2 * q - 1) ** 2)
    # entries that share a row of A or of W are dependent (through the rows' popcounts when
    # p != 0.5), so the standard error of the mean is bounded with 1/m + 1/n, not 1/(m n)
    assert abs(d.mean() - mean) < 6 * np.sqrt(var * (1.0 / m + 1.0 / n))
    assert 0.8 * var < d.var() < 1.25 * var


# ---------------------------------------------------------------- affine + Sign on integers
def test_affine_sign_is_single_rounding_exact_rational():
    rng = np.random.default_rng(0)
    k = 64
    d = np.arange(-k, k + 1, 2, dtype=np.int32)[None, :].repeat(4, 0)
    n = d.shape[1]
    scale = rng.uniform(-1.5, 1.5, n).astype(np.float32)
    scale[:4] = [0.0, -0.0, 1.0, -1.0]
    shift = rng.normal(0, 3.0, n).astype(np.float32)
    shift[4:8] = [0.0, -0.0, 2.0, -2.0]
    scale[6], scale[7] = 1.0, 1.0
    d[:, 6], d[:, 7] = -2, 2          # exact zeros: 1*(-2)+2 and 1*2-2
    for mode in (o.SIGN_ZERO_POS, o.SIGN_ZERO_NEG):
        P, Y = o.affine_sign_pack_i32(d, scale, shift, mode, want_y=True)
        got = o.unpack_pm1(P, n)
        for j in range(n):
            exact = Fraction(float(scale[j])) * int(d[0, j]) + Fraction(float(shift[j]))
            want = 1 if (exact > 0 or (exact == 0 and mode == o.SIGN_ZERO_POS)) else -1
            assert got[0, j] == want, (j, mode)
            assert Y[0, j] == np.float32(float(exact)) or abs(Y[0, j] - float(exact)) <= abs(float(exact)) * 2 ** -23
        assert got[0, 6] == got[0, 7] == (1 if mode == o.SIGN_ZERO_POS else -1)


def test_affine_sign_fma_differs_from_two_roundings():
    """s*d rounded to fp32 and then added to b gives exactly 0 here, the fused form does not."""
    s = np.float32(1.0) + np.float32(2.0 ** -23)
    dval = 3
    prod32 = np.float32(s * np.float32(dval))           # product rounded to fp32
    b = -prod32
    exact = Fraction(float(s)) * dval + Fraction(float(b))
    assert exact != 0 and np.float32(prod32 + b) == 0
    P = o.affine_sign_pack_i32(np.array([[dval]], np.int32), [s], [b], o.SIGN_ZERO_POS)
    assert o.unpack_pm1(P, 1)[0, 0] == (1 if exact > 0 else -1)
    assert exact < 0   # so a two-rounding implementation (0 -> +1) would be caught


def test_affine_sign_defaults_scale1_shift0():
    d = np.array([[-3, 0, 5]], np.int32)
    np.testing.assert_array_equal(o.unpack_pm1(o.affine_sign_pack_i32(d, None, None, o.SIGN_ZERO_NEG), 3),
                                  [[-1, -1, 1]])
    np.testing.assert_array_equal(o.unpack_pm1(o.affine_sign_pack_i32(d, None, None, o.SIGN_ZERO_POS), 3),
                                  [[-1, 1, 1]])


# ---------------------------------------------------------------- +-1 weights x real input
@pytest.mark.parametrize("k", [1, 33, 440])
def test_signw_gemm_against_float64_matmul(k):
    rng = np.random.default_rng(k)
    x = rng.standard_normal((6, k)).astype(np.float32)
    w = wl.make_bit_matrix(11, k, 0.5, [12, k])
    y, sa = o.signw_gemm(x, np_pack(w), k)
    ref = x.astype(np.float64) @ pm1(w).T
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12 * k)
    np.testing.assert_allclose(sa, np.abs(x.astype(np.float64)).sum(1), rtol=1e-14)
    # add/subtract form: y = 2 * sum_{bit=1} x - sum x
    alt = 2 * (x.astype(np.float64)[:, None, :] * w[None, :, :]).sum(-1) - x.astype(np.float64).sum(1)[:, None]
    np.testing.assert_allclose(y, alt, rtol=0, atol=1e-11 * k)


def test_signw_gemm_integer_inputs_exact():
    rng = np.random.default_rng(1)
    x = rng.integers(-8, 9, (4, 70)).astype(np.float32)
    w = wl.make_bit_matrix(5, 70, 0.5, 13)
    y, _ = o.signw_gemm(x, np_pack(w), 70)
    np.testing.assert_array_equal(y, x.astype(np.int64) @ (2 * w.astype(np.int64) - 1).T)


def test_affine_act_f64():
    y = np.array([[-4.0, -0.5, 0.0, 0.5, 4.0]])
    sc = np.array([0.5, 0.5, 1.0, -0.5, 0.5], np.float32)
    sh = np.array([0.0, 0.25, 0.0, 0.0, -2.0], np.float32)
    yh, h, p = o.affine_act_f64(y, sc, sh, o.ACT_HARDTANH)
    np.testing.assert_array_equal(yh, [[-2.0, 0.0, 0.0, -0.25, 0.0]])
    np.testing.assert_array_equal(h, [[-1.0, 0.0, 0.0, -0.25, 0.0]])
    assert p is None
    _, h, p = o.affine_act_f64(y, sc, sh, o.ACT_SIGN, o.SIGN_ZERO_POS)
    np.testing.assert_array_equal(h, [[-1, 1, 1, -1, 1]])
    np.testing.assert_array_equal(o.unpack_pm1(p, 5), [[-1, 1, 1, -1, 1]])
    _, h, p = o.affine_act_f64(y, sc, sh, o.ACT_SIGN, o.SIGN_ZERO_NEG)
    np.testing.assert_array_equal(h, [[-1, -1, -1, -1, -1]])
    _, h, _ = o.affine_act_f64(y, None, None, o.ACT_NONE)
    np.testing.assert_array_equal(h, y)


# ---------------------------------------------------------------- top layer + log-softmax
def test_real_gemm_bits_and_f32_against_matmul():
    rng = np.random.default_rng(2)
    hdim, c = 70, 13
    hb = wl.make_bit_matrix(5, hdim, 0.5, 14)
    wout = rng.standard_normal((c, hdim)).astype(np.float32)
    b = rng.standard_normal(c).astype(np.float32)
    ref = pm1(hb) @ wout.astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_allclose(o.real_gemm_bits(np_pack(hb), wout, b, hdim), ref, atol=1e-12)
    hf = rng.uniform(-1, 1, (5, hdim)).astype(np.float32)
    ref = hf.astype(np.float64) @ wout.astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_allclose(o.real_gemm_f32(hf, wout, b), ref, atol=1e-12)


def test_log_softmax_pins():
    import torch
    rng = np.random.default_rng(3)
    z = rng.standard_normal((9, 3307)) * 5
    lp = o.log_softmax(z)
    np.testing.assert_allclose(np.exp(lp).sum(1), 1.0, atol=1e-12)
    np.testing.assert_allclose(lp, torch.log_softmax(torch.from_numpy(z), dim=1).numpy(), atol=1e-12)
    np.testing.assert_allclose(o.log_softmax(z + 1000.0), lp, atol=1e-9)    # shift invariance
    np.testing.assert_allclose(o.log_softmax(np.zeros((2, 3972))), -np.log(3972.0), atol=1e-13)
    # large spread must not overflow
    big = np.array([[1000.0, 0.0, -1000.0]])
    np.testing.assert_allclose(o.log_softmax(big), [[0.0, -1000.0, -2000.0]], atol=1e-9)


# ---------------------------------------------------------------- whole forward
def numpy_forward_alg2(X, W, r, Wout, bout):
    """Algorithm 2's forward loop with Algorithm 1's weight binarisation, written with
    numpy only, on values for which all arithmetic is exact (integers and halves)."""
    h = X.astype(np.float64)
    for w, b in zip(W, r):
        wb = np.where(w > 0, 1.0, -1.0)
        hh = h @ wb.T + b
        h = np.where(hh > 0, 1.0, -1.0)
    z = h @ Wout.astype(np.float64).T + bout
    z = z - z.max(1, keepdims=True)
    return z - np.log(np.exp(z).sum(1, keepdims=True))


def test_forward_reduces_to_algorithm2_with_unit_scale():
    rng = np.random.default_rng(4)
    dims = [37, 50, 41, 33]
    X = rng.integers(-4, 5, (6, dims[0])).astype(np.float32)
    W = [rng.choice([-0.7, 0.0, 0.3, 1.0], (dims[i + 1], dims[i])).astype(np.float32) for i in range(3)]
    r = [(rng.integers(-3, 4, dims[i + 1]) + 0.5).astype(np.float32) for i in range(3)]
    r[1][:5] = [0.0, 1.0, -1.0, 2.0, -2.0]   # exact zeros can occur: Eq. 3 sends them to -1
    Wout = rng.standard_normal((19, dims[-1])).astype(np.float32)
    bout = rng.standard_normal(19).astype(np.float32)
    t = o.forward(X, W, [None] * 3, r, Wout, bout, o.ACT_SIGN, o.SIGN_ZERO_NEG)
    np.testing.assert_allclose(t["logp"], numpy_forward_alg2(X, W, r, Wout, bout), atol=1e-12)
    # the zero-positive convention changes the result on this input (zeros do occur)
    t2 = o.forward(X, W, [None] * 3, r, Wout, bout, o.ACT_SIGN, o.SIGN_ZERO_POS)
    assert any((a != b).any() for a, b in zip(t["bits"], t2["bits"]))


def test_forward_binary_weight_variant_against_numpy():
    rng = np.random.default_rng(5)
    dims = [20, 30, 25]
    X = rng.standard_normal((4, dims[0])).astype(np.float32)
    W = [rng.standard_normal((dims[i + 1], dims[i])).astype(np.float32) for i in range(2)]
    sc = [np.full(dims[i + 1], a, np.float32) for i, a in enumerate([0.05, 0.08])]
    sh = [np.zeros(dims[i + 1], np.float32) for i in range(2)]
    Wout = rng.standard_normal((7, dims[-1])).astype(np.float32)
    bout = rng.standard_normal(7).astype(np.float32)
    t = o.forward(X, W, sc, sh, Wout, bout, o.ACT_HARDTANH)
    h = X.astype(np.float64)
    for w, s in zip(W, sc):
        h = np.clip((h @ np.where(w >= 0, 1.0, -1.0).T) * s.astype(np.float64), -1, 1)
        h = h.astype(np.float32).astype(np.float64)   # activations are handed on as fp32
    z = h @ Wout.astype(np.float64).T + bout
    z = z - z.max(1, keepdims=True)
    np.testing.assert_allclose(t["logp"], z - np.log(np.exp(z).sum(1, keepdims=True)), atol=1e-12)


# ---------------------------------------------------------------- (0,1) activations (Section 3.2)
@pytest.mark.parametrize("k", [1, 31, 32, 33, 127, 440, 600])
def test_gemm01_brute_force_float_matmul(k):
    h = wl.make_bit_matrix(5, k, 0.4, [12, k])
    w = wl.make_bit_matrix(9, k, 0.5, [13, k])
    d = o.gemm01(np_pack(h), np_pack(w), k)
    ref = h.astype(np.float64) @ pm1(w).T   # h in {0,1}, w in {-1,+1}; exact in float64
    assert d.dtype == np.int32 and d.shape == (5, 9)
    np.testing.assert_array_equal(d, ref.astype(np.int64))


def test_gemm01_invariants_and_relation_to_the_pm1_product():
    k = 203
    h = wl.make_bit_matrix(6, k, 0.5, 21)
    w = wl.make_bit_matrix(4, k, 0.3, 22)
    hp, wp = np_pack(h), np_pack(w)
    d = o.gemm01(hp, wp, k)
    ones = h.sum(1, dtype=np.int64)
    # |d| <= number of ones in the row, and d has that number's parity
    assert np.all(np.abs(d) <= ones[:, None]) and np.all((d - ones[:, None]) % 2 == 0)
    # AND-popcount identity  d = 2 popc(h and w) - popc(h)
    an = (h[:, None, :] & w[None, :, :]).sum(-1).astype(np.int64)
    np.testing.assert_array_equal(d, 2 * an - ones[:, None])
    # h = (a + 1) / 2  =>  2 d = dot_pm1(a, w) + sum_k w[n][k]
    wsum = pm1(w).sum(1).astype(np.int64)
    np.testing.assert_array_equal(2 * d, o.xnor_gemm(hp, wp, k) + wsum[None, :])
    # an all-zero row gives 0, an all-one row the sum of the unit's weights
    np.testing.assert_array_equal(o.gemm01(np_pack(np.zeros((1, k), np.uint8)), wp, k), 0)
    np.testing.assert_array_equal(o.gemm01(np_pack(np.ones((1, k), np.uint8)), wp, k)[0], wsum)
    # pad bits and pitch words are ignored
    hp2 = np.concatenate([hp, np.full((6, 2), 0xFFFFFFFF, np.uint32)], 1)
    hp2[:, (k - 1) // 32] |= np.uint32((0xFFFFFFFF << (k % 32)) & 0xFFFFFFFF)
    np.testing.assert_array_equal(o.gemm01(hp2, wp, k), d)


def test_real_gemm_bits01_against_matmul():
    rng = np.random.default_rng(8)
    h = wl.make_bit_matrix(7, 70, 0.5, 31)
    Wout = rng.standard_normal((11, 70)).astype(np.float32)
    b = rng.standard_normal(11).astype(np.float32)
    z = o.real_gemm_bits01(np_pack(h), Wout, b, 70)
    np.testing.assert_allclose(z, h.astype(np.float64) @ Wout.astype(np.float64).T + b, atol=1e-12)


def test_forward_with_01_activations_against_numpy():
    """Algorithm 2's forward loop with the hidden activations in (0,1): h = 1 where the
    pre-activation is positive, 0 elsewhere; exactly representable values, so the numpy
    restatement must agree to rounding."""
    rng = np.random.default_rng(14)
    dims = [37, 50, 41, 33]
    X = rng.integers(-4, 5, (6, dims[0])).astype(np.float32)
    W = [rng.choice([-0.7, 0.0, 0.3, 1.0], (dims[i + 1], dims[i])).astype(np.float32) for i in range(3)]
    r = [(rng.integers(-3, 4, dims[i + 1]) + 0.5).astype(np.float32) for i in range(3)]
    r[1][:5] = [0.0, 1.0, -1.0, 2.0, -2.0]
    Wout = rng.standard_normal((19, dims[-1])).astype(np.float32)
    bout = rng.standard_normal(19).astype(np.float32)
    t = o.forward(X, W, [None] * 3, r, Wout, bout, o.ACT_SIGN, o.SIGN_ZERO_NEG, values=o.VALUES_01)
    h = X.astype(np.float64)
    for w, b in zip(W, r):
        wb = np.where(w > 0, 1.0, -1.0)                  # Eq. 3 as printed
        h = ((h @ wb.T + b.astype(np.float64)) > 0).astype(np.float64)
    z = h @ Wout.astype(np.float64).T + bout
    z = z - z.max(1, keepdims=True)
    np.testing.assert_allclose(t["logp"], z - np.log(np.exp(z).sum(1, keepdims=True)), atol=1e-12)
    # and it is a different function from the (-1,+1) network on this input
    t2 = o.forward(X, W, [None] * 3, r, Wout, bout, o.ACT_SIGN, o.SIGN_ZERO_NEG)
    assert np.abs(t["logp"] - t2["logp"]).max() > 1e-3


# ---------------------------------------------------------------- front and back of a hybrid model
def test_splice_context_window():
    """The 11-frame context of Section 3: interior rows are plain concatenations of the
    neighbouring frames, edges repeat the first / last frame, no context is the identity."""
    rng = np.random.default_rng(3)
    F = rng.standard_normal((9, 4)).astype(np.float32)
    np.testing.assert_array_equal(o.splice(F, 0, 0), F)
    S = o.splice(F, 2, 1)
    assert S.shape == (9, 16)
    np.testing.assert_array_equal(S[4], np.concatenate([F[2], F[3], F[4], F[5]]))
    np.testing.assert_array_equal(S[0], np.concatenate([F[0], F[0], F[0], F[1]]))
    np.testing.assert_array_equal(S[1], np.concatenate([F[0], F[0], F[1], F[2]]))
    np.testing.assert_array_equal(S[8], np.concatenate([F[6], F[7], F[8], F[8]]))
    # the same window through numpy's own edge padding
    P = np.pad(F, ((2, 1), (0, 0)), mode="edge")
    np.testing.assert_array_equal(S, np.concatenate([P[t:t + 9] for t in range(4)], axis=1))
    # a window longer than the matrix still only repeats existing rows
    one = o.splice(F[:1], 5, 5)
    np.testing.assert_array_equal(one, np.tile(F[:1], (1, 11)))


def test_forward_log_prior_is_subtracted_from_log_posteriors():
    rng = np.random.default_rng(6)
    dims = [12, 20, 16]
    X = rng.standard_normal((5, dims[0])).astype(np.float32)
    W = [rng.standard_normal((dims[i + 1], dims[i])).astype(np.float32) for i in range(2)]
    sc = [np.ones(dims[i + 1], np.float32) for i in range(2)]
    sh = [np.zeros(dims[i + 1], np.float32) for i in range(2)]
    Wout = rng.standard_normal((7, dims[-1])).astype(np.float32)
    bout = rng.standard_normal(7).astype(np.float32)
    prior = rng.dirichlet(np.ones(7))
    lp = np.log(prior).astype(np.float32)
    a = o.forward(X, W, sc, sh, Wout, bout)
    b = o.forward(X, W, sc, sh, Wout, bout, log_prior=lp)
    np.testing.assert_allclose(b["logp"], a["logp"] - lp.astype(np.float64)[None, :], atol=1e-12)
    # posterior / prior, summed with the prior as weights, is 1 again
    np.testing.assert_allclose((np.exp(b["logp"]) * np.exp(lp.astype(np.float64))).sum(1), 1.0, atol=1e-9)


# ---------------------------------------------------------------- Sigmoid layers, mixed topology
def test_sigmoid_activation_pins():
    from scipy.special import expit
    y = np.array([[0.0, 1.0, -1.0, 30.0, -30.0, 1e-3, -745.0, 710.0]])
    _, H, _ = o.affine_act_f64(y, None, None, o.ACT_SIGMOID)
    np.testing.assert_allclose(H, expit(y), rtol=1e-15, atol=0)
    assert H[0, 0] == 0.5
    np.testing.assert_allclose(H[0, 1] + H[0, 2], 1.0, atol=1e-16)   # sigma(-x) = 1 - sigma(x)
    # integer dot products through the fp32 affine
    d = np.array([[-5, 0, 3, 100]], dtype=np.int32)
    sc = np.array([0.5, 1.0, -2.0, 0.25], dtype=np.float32)
    sh = np.array([0.25, 0.0, 1.0, -25.0], dtype=np.float32)
    np.testing.assert_allclose(o.affine_sigmoid_i32(d, sc, sh), expit(np.array([[-2.25, 0.0, -5.0, 0.0]])), rtol=1e-15)


def test_forward_mixed_topology_against_numpy():
    """(Sigmoid, Sign, Sign, Sigmoid, Softmax) with real first-layer and Softmax weights, written
    again with numpy on values whose layer-2 pre-activations are far from zero."""
    from scipy.special import expit
    rng = np.random.default_rng(12)
    dims = [23, 40, 36, 32, 28]
    X = rng.standard_normal((7, dims[0])).astype(np.float32)
    W = [rng.standard_normal((dims[i + 1], dims[i])).astype(np.float32) for i in range(4)]
    sc = [None] + [rng.uniform(0.5, 1.5, dims[i + 1]).astype(np.float32) for i in range(1, 4)]
    sh = [rng.standard_normal(dims[i + 1]).astype(np.float32) * 0.3 for i in range(4)]
    Wout = rng.standard_normal((9, dims[-1])).astype(np.float32)
    bout = rng.standard_normal(9).astype(np.float32)
    t = o.forward_mixed(X, W, sc, sh, Wout, bout, o.SIGN_ZERO_NEG)
    f64 = lambda a: a.astype(np.float64)
    h = expit(f64(X) @ f64(W[0]).T + f64(sh[0])).astype(np.float32)
    y = (f64(h) @ np.where(W[1] > 0, 1.0, -1.0).T) * f64(sc[1]) + f64(sh[1])
    assert np.abs(y).min() > 1e-6
    a = np.where(y > 0, 1.0, -1.0)
    d = a @ np.where(W[2] > 0, 1.0, -1.0).T
    a = np.where((np.float32(1) * (sc[2] * d.astype(np.float32) + sh[2])) > 0, 1.0, -1.0)
    d = a @ np.where(W[3] > 0, 1.0, -1.0).T
    hL = expit(f64((sc[3] * d.astype(np.float32) + sh[3]).astype(np.float32))).astype(np.float32)
    z = f64(hL) @ f64(Wout).T + f64(bout)
    z = z - z.max(1, keepdims=True)
    want = z - np.log(np.exp(z).sum(1, keepdims=True))
    # two roundings instead of one fma can move a value by an ulp: far inside the tolerance
    np.testing.assert_allclose(t["logp"], want, atol=1e-5)
    np.testing.assert_array_equal(o.unpack_pm1(t["bits"][0], dims[2]), np.where(y > 0, 1, -1))
