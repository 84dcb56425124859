"""Parity of the CUDA path (called through the C ABI) with the CPU oracle, element by
element on the same seeded inputs.  Integers and packed bits must be bit-exact; floats
within 1e-4 * sum|x_i| per output (first-layer / sign-weight GEMM) and 1e-4 absolute on
log-probabilities."""
import numpy as np
import pytest

from oracle import bnn_oracle as o
from paper_1706_09453_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FLOAT_TOL = 1e-4   # x sum_k |x[m][k]| per output
LOGP_TOL = 1e-4    # absolute, on log-probabilities


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_1706_09453_b200 import build, binding
    build.build()
    return binding


@pytest.fixture(scope="module")
def torch_():
    import torch
    return torch


@pytest.fixture(params=["popc", "tensor", "prepared"])
def xnor_path(request, B):
    """Runs a test once per XNOR kernel: integer-pipe popcount, tcgen05 tensor core widening both
    operands on the fly, tcgen05 with the weights widened once (bnn_xnor_prepare)."""
    prev = B.bnn_set_xnor_path(B.XNOR_POPC if request.param == "popc" else B.XNOR_TENSOR)
    yield request.param
    B.bnn_set_xnor_path(prev)
    assert B.bnn_device_status() == 0, "a tensor-core kernel gave up on a bounded wait"


def run_xnor(B, path, a_dev, w_dev, k, image=None, **kw):
    """bnn_xnor_gemm, or (path "prepared") bnn_xnor_prepare + bnn_xnor_gemm_prepared."""
    if path != "prepared":
        return B.bnn_xnor_gemm(a_dev, w_dev, k, **kw)
    import torch
    n = w_dev.shape[0]
    if image is None:
        image = torch.full((B.bnn_xnor_prepared_bytes(n, k),), 0x5A, dtype=torch.uint8, device="cuda:0")
        B.bnn_xnor_prepare(w_dev, k, image)
    B.bnn_xnor_gemm_prepared(a_dev, image, n, k, **kw)
    return image


@pytest.fixture(params=["fp32", "tensor", "tensor_ws"])
def real_path(request, B):
    """Runs a test once per real-valued GEMM kernel: FP32 pipe, tcgen05 with operands split on
    the fly, tcgen05 with the activations split once into scratch (tensor_ws)."""
    prev = B.bnn_set_option(B.OPT_REAL_PATH, B.PATH_CUDA_CORE if request.param == "fp32" else B.PATH_TENSOR)
    yield request.param
    B.bnn_set_option(B.OPT_REAL_PATH, prev)
    assert B.bnn_device_status() == 0, "a tensor-core kernel gave up on a bounded wait"


def signw_ws(B, path, m, k):
    """Scratch for bnn_signw_gemm_ws when the test runs the split-once path, else None."""
    if path != "tensor_ws":
        return None
    import torch
    return torch.empty(B.bnn_signw_workspace_bytes(m, k) + 256, dtype=torch.uint8, device="cuda:0")


def dev(a):
    from paper_1706_09453_b200.model import to_dev
    return to_dev(a)


def host_words(t, k):
    from paper_1706_09453_b200.model import words_to_numpy
    return words_to_numpy(t, k)


def packed_canary(torch, rows, k, B, fill=0x5A5A5A5A):
    return torch.full((rows, B.packed_pitch(k) + 4), fill, dtype=torch.int32, device="cuda:0")


# ------------------------------------------------------------------ Sign + pack (Eq. 3)
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("shape", [(1, 1), (3, 31), (5, 32), (7, 33), (9, 127), (130, 440), (257, 600), (64, 2048)])
def test_pack_matches_oracle(B, torch_, mode, shape):
    m, k = shape
    rng = np.random.default_rng(m * 1000 + k)
    x = rng.standard_normal((m, k + 3)).astype(np.float32)   # pitch k+3: rows not 16-byte aligned
    x[rng.random(x.shape) < 0.1] = 0.0
    x[0, 0] = -0.0
    if k > 4:
        x[0, 1], x[0, 2], x[0, 3], x[0, 4] = np.nan, np.float32(1e-45), -np.float32(1e-45), np.inf
    xd = dev(x)[:, :k]
    out = packed_canary(torch_, m, k, B)
    view = out[:, :B.packed_pitch(k)]
    (B.bnn_binarize_pack if m % 2 else B.bnn_pack_weights)(xd, view, mode)
    torch_.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint32)
    kw = (k + 31) // 32
    np.testing.assert_array_equal(got[:, :kw], o.sign_pack(x[:, :k], mode))
    np.testing.assert_array_equal(got[:, kw:], 0x5A5A5A5A)   # pitch words untouched


def test_pack_vectorised_path_aligned_rows(B, torch_):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((300, 440)).astype(np.float32)
    out = packed_canary(torch_, 300, 440, B)
    B.bnn_binarize_pack(dev(x), out[:, :16], 0)
    got = out.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got[:, :14], o.sign_pack(x, 0))
    np.testing.assert_array_equal(got[:, 14:], 0x5A5A5A5A)


# ------------------------------------------------------------------ threshold fold
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("k", [1, 64, 441])
def test_fold_thresholds_exhaustive(B, torch_, mode, k):
    """(d >= thr) xor flip == Sign(fma(scale, d, shift)) for EVERY integer d in [-K, K]."""
    rng = np.random.default_rng(k)
    n = 200
    scale = rng.uniform(-1.5, 1.5, n).astype(np.float32)
    shift = rng.normal(0, 0.3 * k, n).astype(np.float32)
    scale[:8] = [0.0, -0.0, 1.0, -1.0, 1e-30, -1e-30, 1e30, -1e30]
    shift[:4] = [0.0, -0.0, 0.0, 0.0]
    shift[8:12] = [1e30, -1e30, float(k), -float(k)]
    scale[12:16] = [1.0, 1.0, -1.0, -1.0]
    shift[12:16] = [2.0, -2.0, 2.0, -2.0]      # exact zeros at d = -+2
    s = np.float32(1.0) + np.float32(2.0 ** -23)
    scale[16], shift[16] = s, -np.float32(s * np.float32(3))   # fma vs two roundings
    thr = torch_.empty(n, dtype=torch_.int32, device="cuda:0")
    flip = torch_.empty((n + 31) // 32, dtype=torch_.int32, device="cuda:0")
    B.bnn_fold_thresholds(dev(scale), dev(shift), n, k, thr, flip, mode)
    thr = thr.cpu().numpy().astype(np.int64)
    fw = flip.cpu().numpy().view(np.uint32)
    fb = ((fw[np.arange(n) // 32] >> (np.arange(n) % 32).astype(np.uint32)) & 1).astype(bool)
    d = np.arange(-k, k + 1, dtype=np.int32)
    D = np.repeat(d[:, None], n, 1)
    want = o.unpack_pm1(o.affine_sign_pack_i32(D, scale, shift, mode), n) == 1
    got = (D >= thr[None, :]) ^ fb[None, :]
    np.testing.assert_array_equal(got, want)


def test_fold_thresholds_null_scale_shift(B, torch_):
    thr = torch_.empty(40, dtype=torch_.int32, device="cuda:0")
    flip = torch_.empty(2, dtype=torch_.int32, device="cuda:0")
    B.bnn_fold_thresholds(None, None, 40, 100, thr, flip, 0)
    assert (thr.cpu().numpy() == 0).all() and (flip.cpu().numpy() == 0).all()
    B.bnn_fold_thresholds(None, None, 40, 100, thr, flip, 1)
    assert (thr.cpu().numpy() == 1).all()


# ------------------------------------------------------------------ XNOR GEMM
XNOR_SHAPES = [(1, 1, 1), (2, 3, 31), (5, 7, 32), (17, 9, 33), (129, 130, 127), (300, 257, 1000),
               (256, 1024, 1024), (131, 1024, 440), (200, 129, 600), (640, 384, 2048), (100, 520, 4100),
               (20000, 256, 96)]


@pytest.mark.parametrize("shape", XNOR_SHAPES)
@pytest.mark.parametrize("p", [0.5, 0.1])
def test_xnor_gemm_int32_bit_exact(B, torch_, xnor_path, shape, p):
    m, n, k = shape
    ap = wl.make_bit_planes(m, k, p, [1, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, p, [2, m, n, k], B.packed_pitch(k))
    c = torch_.full((m, n + 5), -77, dtype=torch_.int32, device="cuda:0")
    run_xnor(B, xnor_path, dev(ap), dev(wp), k, C_out=c[:, :n])
    got = c.cpu().numpy()
    np.testing.assert_array_equal(got[:, :n], o.xnor_gemm(ap, wp, k))
    np.testing.assert_array_equal(got[:, n:], -77)


@pytest.mark.parametrize("shape", [(96, 40, 8192), (65536, 24, 1024)])
def test_xnor_gemm_int32_longest_fan_in_and_largest_batch(B, torch_, xnor_path, shape):
    """The corner sizes of the GEMM sweep (fan-in 8192; 65536 frames) with few units, so that the
    oracle checks every output: all three kernels, every element."""
    m, n, k = shape
    ap = wl.make_bit_planes(m, k, 0.5, [5, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, 0.1, [6, m, n, k], B.packed_pitch(k))
    c = torch_.full((m, n), -77, dtype=torch_.int32, device="cuda:0")
    run_xnor(B, xnor_path, dev(ap), dev(wp), k, C_out=c)
    np.testing.assert_array_equal(c.cpu().numpy(), o.xnor_gemm(ap, wp, k))
    assert B.bnn_device_status() == 0


def test_xnor_prepared_right_after_its_setup_on_one_stream(B, torch_):
    """Thresholds folded, weights prepared and the fused layer launched back to back on one stream,
    several times over with changing parameters: the layer must see each set-up's results (plain
    stream order is all the header promises)."""
    m, n, k = 1000, 384, 2048
    rng = np.random.default_rng(5)
    ap = wl.make_bit_planes(m, k, 0.5, [7, m, n, k], B.packed_pitch(k))
    a_dev = dev(ap)
    thr = torch_.zeros(n, dtype=torch_.int32, device="cuda:0")
    flip = torch_.zeros((n + 31) // 32, dtype=torch_.int32, device="cuda:0")
    image = torch_.empty(B.bnn_xnor_prepared_bytes(n, k), dtype=torch_.uint8, device="cuda:0")
    out = torch_.zeros((m, B.packed_pitch(n)), dtype=torch_.int32, device="cuda:0")
    for rep in range(4):
        wp = wl.make_bit_planes(n, k, 0.5, [8, rep, n, k], B.packed_pitch(k))
        scale = rng.uniform(0.5, 1.5, n).astype(np.float32) * (1 if rep % 2 else -1)
        shift = rng.normal(0, 3.0, n).astype(np.float32)
        w_dev, sc, sh = dev(wp), dev(scale), dev(shift)
        B.bnn_fold_thresholds(sc, sh, n, k, thr, flip, 0)
        B.bnn_xnor_prepare(w_dev, k, image)
        B.bnn_xnor_gemm_prepared(a_dev, image, n, k, thr=thr, flip=flip, out_bits=out)
        want = o.affine_sign_pack_i32(o.xnor_gemm(ap, wp, k), scale, shift, 0)
        np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32)[:, :(n + 31) // 32], want)
    assert B.bnn_device_status() == 0


def test_xnor_gemm_ignores_garbage_in_pad_bits(B, torch_, xnor_path):
    m, n, k = 70, 90, 1000 - 13
    pitch = B.packed_pitch(k) + 4
    ap = wl.make_bit_planes(m, k, 0.5, 11, pitch)
    wp = wl.make_bit_planes(n, k, 0.5, 12, pitch)
    want = o.xnor_gemm(ap, wp, k)
    kw = (k + 31) // 32
    rng = np.random.default_rng(0)
    ap2, wp2 = ap.copy(), wp.copy()
    ap2[:, kw:] = rng.integers(0, 2**32, (m, pitch - kw), dtype=np.uint32)
    wp2[:, kw:] = rng.integers(0, 2**32, (n, pitch - kw), dtype=np.uint32)
    ap2[:, kw - 1] |= np.uint32(0xFFFFFFFF << (k % 32) & 0xFFFFFFFF)
    wp2[:, kw - 1] |= rng.integers(0, 2**32, n, dtype=np.uint32) & np.uint32(0xFFFFFFFF << (k % 32) & 0xFFFFFFFF)
    c = torch_.empty((m, n), dtype=torch_.int32, device="cuda:0")
    run_xnor(B, xnor_path, dev(ap2), dev(wp2), k, C_out=c)
    np.testing.assert_array_equal(c.cpu().numpy(), want)


@pytest.mark.parametrize("shape", [(5, 7, 33), (129, 130, 127), (300, 257, 1000), (256, 1024, 1024), (131, 96, 440),
                                   (19100, 300, 160), (300, 260, 3000), (150, 200, 5000), (2000, 3072, 2100)])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("with_c", [False, True])
def test_xnor_gemm_fused_sign_pack_bit_exact(B, torch_, xnor_path, shape, mode, with_c):
    m, n, k = shape
    rng = np.random.default_rng(m + n + k)
    ap = wl.make_bit_planes(m, k, 0.5, [3, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, 0.5, [4, m, n, k], B.packed_pitch(k))
    scale = rng.uniform(0.5, 1.5, n).astype(np.float32)
    shift = rng.normal(0, 0.1, n).astype(np.float32)
    scale[::7] *= -1                      # negative scales flip the comparison
    scale[1::11] = 0.0
    shift[2::5] = np.round(shift[2::5] * 20)   # integer shifts with scale...
    scale[2::5] = 1.0                          # ... 1 make exact zeros likely
    thr = torch_.empty(n, dtype=torch_.int32, device="cuda:0")
    flip = torch_.empty((n + 31) // 32, dtype=torch_.int32, device="cuda:0")
    B.bnn_fold_thresholds(dev(scale), dev(shift), n, k, thr, flip, mode)
    out = packed_canary(torch_, m, n, B)
    c = torch_.empty((m, n), dtype=torch_.int32, device="cuda:0") if with_c else None
    run_xnor(B, xnor_path, dev(ap), dev(wp), k, C_out=c, thr=thr, flip=flip, out_bits=out[:, :B.packed_pitch(n)])
    d = o.xnor_gemm(ap, wp, k)
    want = o.affine_sign_pack_i32(d, scale, shift, mode)
    got = out.cpu().numpy().view(np.uint32)
    nw = (n + 31) // 32
    np.testing.assert_array_equal(got[:, :nw], want)
    np.testing.assert_array_equal(got[:, nw:], 0x5A5A5A5A)
    if with_c:
        np.testing.assert_array_equal(c.cpu().numpy(), d)
    if mode == 0 and m * n > 100000:
        assert (d[:, 2::5].astype(np.float32) + shift[2::5] == 0).any(), "no exact zero was exercised"


@pytest.mark.parametrize("path", ["tensor", "prepared"])
@pytest.mark.parametrize("shape", [(8192, 2048, 2048), (16384, 2048, 2048)])
def test_xnor_gemm_full_size_every_output_on_repeated_launches(B, torch_, shape, path):
    """A hidden layer at full size, every output bit compared with the oracle, on many launches in
    a row: a hand-off between the kernel's roles that is wrong once in ten thousand tiles only
    shows on a run of this length (sampled outputs would miss it)."""
    m, n, k = shape
    prev = B.bnn_set_xnor_path(B.XNOR_TENSOR)
    try:
        rng = np.random.default_rng(m)
        ap = wl.make_bit_planes(m, k, 0.5, [5, m, n, k], B.packed_pitch(k))
        wp = wl.make_bit_planes(n, k, 0.5, [6, m, n, k], B.packed_pitch(k))
        scale = np.ones(n, dtype=np.float32)
        shift = np.round(rng.normal(0, 20, n)).astype(np.float32)   # thresholds where the dot products are dense
        thr = torch_.empty(n, dtype=torch_.int32, device="cuda:0")
        flip = torch_.empty((n + 31) // 32, dtype=torch_.int32, device="cuda:0")
        B.bnn_fold_thresholds(dev(scale), dev(shift), n, k, thr, flip, 0)
        d = o.xnor_gemm(ap, wp, k)
        want_bits = torch_.from_numpy(o.affine_sign_pack_i32(d, scale, shift, 0).view(np.int32)).to("cuda:0")
        want_c = torch_.from_numpy(d).to("cuda:0")
        a_dev, w_dev = dev(ap), dev(wp)
        out = torch_.zeros((m, B.packed_pitch(n)), dtype=torch_.int32, device="cuda:0")
        c = torch_.zeros((m, n), dtype=torch_.int32, device="cuda:0")
        nw = (n + 31) // 32
        image = None
        for launch in range(40):
            out.zero_()
            image = run_xnor(B, path, a_dev, w_dev, k, image=image, thr=thr, flip=flip, out_bits=out)
            bad = int((out[:, :nw] != want_bits).sum().item())
            assert bad == 0, "launch %d (fused Sign): %d packed words differ" % (launch, bad)
        for launch in range(20):
            c.zero_()
            run_xnor(B, path, a_dev, w_dev, k, image=image, C_out=c)
            bad = int((c != want_c).sum().item())
            assert bad == 0, "launch %d (int32 output): %d outputs differ" % (launch, bad)
    finally:
        B.bnn_set_xnor_path(prev)
    assert B.bnn_device_status() == 0, "a tensor-core kernel gave up on a bounded wait"


# ------------------------------------------------------------------ (0,1) activations (Section 3.2)
def run_gemm01(B, path, h_dev, w_dev, k, **kw):
    """bnn_gemm01 with packed weights, or (path "prepared") with their prepared image only."""
    if path != "prepared":
        return B.bnn_gemm01(h_dev, w_dev, k, **kw)
    import torch
    n = w_dev.shape[0]
    image = torch.empty(B.bnn_xnor_prepared_bytes(n, k), dtype=torch.uint8, device="cuda:0")
    B.bnn_xnor_prepare(w_dev, k, image)
    B.bnn_gemm01(h_dev, None, k, N=n, prepared=image, **kw)


@pytest.mark.parametrize("shape", [(1, 1, 1), (5, 7, 33), (129, 130, 127), (300, 257, 1000), (256, 1024, 1024),
                                   (131, 1024, 440), (100, 520, 4100), (700, 200, 3000)])
@pytest.mark.parametrize("p", [0.5, 0.1])
def test_gemm01_int32_bit_exact(B, torch_, xnor_path, shape, p):
    m, n, k = shape
    hp = wl.make_bit_planes(m, k, p, [7, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, 0.5, [8, m, n, k], B.packed_pitch(k))
    # garbage in the pad bits of the frame operand must not count as ones
    kw = (k + 31) // 32
    hp_dirty = hp.copy()
    if k % 32:
        hp_dirty[:, kw - 1] |= np.uint32((0xFFFFFFFF << (k % 32)) & 0xFFFFFFFF)
    hp_dirty[:, kw:] = 0xFFFFFFFF
    c = torch_.full((m, n + 5), -77, dtype=torch_.int32, device="cuda:0")
    run_gemm01(B, xnor_path, dev(hp_dirty), dev(wp), k, C_out=c[:, :n])
    got = c.cpu().numpy()
    np.testing.assert_array_equal(got[:, :n], o.gemm01(hp, wp, k))
    np.testing.assert_array_equal(got[:, n:], -77)


@pytest.mark.parametrize("shape", [(5, 7, 33), (300, 257, 1000), (256, 1024, 1024), (2100, 2048, 2048), (700, 200, 3000),
                                   (150, 200, 5000)])
@pytest.mark.parametrize("mode", [0, 1])
def test_gemm01_fused_sign_pack_bit_exact(B, torch_, xnor_path, shape, mode):
    m, n, k = shape
    rng = np.random.default_rng(m + n + k)
    hp = wl.make_bit_planes(m, k, 0.5, [9, m, n, k], B.packed_pitch(k))
    wp = wl.make_bit_planes(n, k, 0.5, [10, m, n, k], B.packed_pitch(k))
    scale = rng.uniform(0.5, 1.5, n).astype(np.float32)
    shift = rng.normal(0, 0.1, n).astype(np.float32)
    scale[::7] *= -1
    shift[2::5] = np.round(shift[2::5] * 20)
    scale[2::5] = 1.0
    thr = torch_.empty(n, dtype=torch_.int32, device="cuda:0")
    flip = torch_.empty((n + 31) // 32, dtype=torch_.int32, device="cuda:0")
    B.bnn_fold_thresholds(dev(scale), dev(shift), n, k, thr, flip, mode)
    out = packed_canary(torch_, m, n, B)
    run_gemm01(B, xnor_path, dev(hp), dev(wp), k, thr=thr, flip=flip, out_bits=out[:, :B.packed_pitch(n)])
    want = o.affine_sign_pack_i32(o.gemm01(hp, wp, k), scale, shift, mode)
    got = out.cpu().numpy().view(np.uint32)
    nw = (n + 31) // 32
    np.testing.assert_array_equal(got[:, :nw], want)
    np.testing.assert_array_equal(got[:, nw:], 0x5A5A5A5A)


@pytest.mark.parametrize("c,m,h", [(2000, 70, 1024), (300, 1100, 1000), (129, 513, 33)])
def test_output_layer_01_activations(B, torch_, real_path, c, m, h):
    rng = np.random.default_rng(c + 1)
    hp = wl.make_bit_planes(m, h, 0.5, 41, B.packed_pitch(h))
    wout = rng.normal(0, 1 / np.sqrt(h), (c, h)).astype(np.float32)
    b = rng.normal(0, 0.1, c).astype(np.float32)
    prep = None
    if real_path != "fp32":
        prep = torch_.empty(B.bnn_output_prepared_bytes(c, h), dtype=torch_.uint8, device="cuda:0")
        B.bnn_output_prepare(dev(wout), prep)
    z = torch_.empty((m, c), dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), z, h, Hp=dev(hp), log_softmax=False, prepared=prep, values=B.VALUES_01)
    zr = o.real_gemm_bits01(hp, wout, b, h)
    assert np.abs(z.cpu().numpy() - zr).max() <= FLOAT_TOL * h
    lp = torch_.empty((m, c), dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), lp, h, Hp=dev(hp), prepared=prep, values=B.VALUES_01)
    assert np.abs(lp.cpu().numpy() - o.log_softmax(zr)).max() <= LOGP_TOL


# ------------------------------------------------------------------ +-1 weights x real input
@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 33), (130, 129, 440), (257, 300, 600), (64, 256, 2048),
                                   (20000, 260, 70), (300, 1300, 100)])
def test_signw_gemm_within_tolerance(B, torch_, real_path, shape):
    m, n, k = shape
    rng = np.random.default_rng(m * n + k)
    x = rng.standard_normal((m, k)).astype(np.float32)
    w = rng.standard_normal((n, k)).astype(np.float32)
    wp = o.sign_pack(w, 0, B.packed_pitch(k))
    y = torch_.full((m, n + 3), 123.0, dtype=torch_.float32, device="cuda:0")
    B.bnn_signw_gemm(dev(x), dev(wp), k, Y=y[:, :n], workspace=signw_ws(B, real_path, m, k))
    got = y.cpu().numpy()
    ref, sumabs = o.signw_gemm(x, wp, k)
    err = np.abs(got[:, :n] - ref)
    assert (err <= FLOAT_TOL * sumabs[:, None]).all(), err.max()
    np.testing.assert_array_equal(got[:, n:], 123.0)


@pytest.mark.parametrize("mode", [0, 1])
def test_signw_gemm_sign_pack_epilogue(B, torch_, real_path, mode):
    m, n, k = 200, 300, 440
    rng = np.random.default_rng(9)
    x = rng.standard_normal((m, k)).astype(np.float32)
    wp = wl.make_bit_planes(n, k, 0.5, 21, B.packed_pitch(k))
    scale = rng.uniform(0.5, 1.5, n).astype(np.float32)
    scale[::9] *= -1
    shift = rng.normal(0, 0.1, n).astype(np.float32)
    out = packed_canary(torch_, m, n, B)
    y = torch_.empty((m, n), dtype=torch_.float32, device="cuda:0")
    B.bnn_signw_gemm(dev(x), dev(wp), k, Y=y, act=B.ACT_SIGN_PACK, scale=dev(scale), shift=dev(shift),
                     out_bits=out[:, :B.packed_pitch(n)], sign_mode=mode, workspace=signw_ws(B, real_path, m, k))
    ref, sumabs = o.signw_gemm(x, wp, k)
    yh, _, bits = o.affine_act_f64(ref, scale, shift, o.ACT_SIGN, mode)
    tol = FLOAT_TOL * np.abs(scale)[None, :] * sumabs[:, None]
    assert (np.abs(y.cpu().numpy() - yh) <= tol + 1e-6).all()
    got = out.cpu().numpy().view(np.uint32)
    nw = (n + 31) // 32
    gs, ws = o.unpack_pm1(got[:, :nw], n), o.unpack_pm1(bits, n)
    decided = np.abs(yh) > tol          # outside the band the bit is determined
    np.testing.assert_array_equal(gs[decided], ws[decided])
    assert decided.mean() > 0.99
    np.testing.assert_array_equal(got[:, nw:], 0x5A5A5A5A)
    # the bits are exactly the Sign of the fp32 values the kernel itself reports
    yv = y.cpu().numpy()
    own = np.where((yv > 0) if mode == 1 else (yv >= 0), 1, -1)
    np.testing.assert_array_equal(gs, own)


def test_signw_gemm_exact_zero_follows_sign_mode(B, torch_, real_path):
    """Integer-valued inputs make y exactly 0 for some units; the bit must follow the mode."""
    m, n, k = 40, 64, 64
    rng = np.random.default_rng(3)
    x = rng.integers(-2, 3, (m, k)).astype(np.float32)
    wp = wl.make_bit_planes(n, k, 0.5, 22, B.packed_pitch(k))
    ref, _ = o.signw_gemm(x, wp, k)
    assert (ref == 0).any()
    for mode in (0, 1):
        out = packed_canary(torch_, m, n, B)
        B.bnn_signw_gemm(dev(x), dev(wp), k, act=B.ACT_SIGN_PACK, out_bits=out[:, :4], sign_mode=mode,
                         workspace=signw_ws(B, real_path, m, k))
        _, _, bits = o.affine_act_f64(ref, None, None, o.ACT_SIGN, mode)
        np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32)[:, :2], bits)


def test_signw_gemm_hardtanh_epilogue(B, torch_, real_path):
    m, n, k = 150, 200, 2048
    rng = np.random.default_rng(4)
    x = rng.uniform(-1, 1, (m, k)).astype(np.float32)
    wp = wl.make_bit_planes(n, k, 0.5, 23, B.packed_pitch(k))
    scale = np.full(n, 0.05, np.float32)
    y = torch_.empty((m, n), dtype=torch_.float32, device="cuda:0")
    B.bnn_signw_gemm(dev(x), dev(wp), k, Y=y, act=B.ACT_HARDTANH, scale=dev(scale), workspace=signw_ws(B, real_path, m, k))
    ref, sumabs = o.signw_gemm(x, wp, k)
    _, h, _ = o.affine_act_f64(ref, scale, None, o.ACT_HARDTANH)
    got = y.cpu().numpy()
    assert (np.abs(got - h) <= FLOAT_TOL * 0.05 * sumabs[:, None]).all()
    assert got.min() >= -1.0 and got.max() <= 1.0 and (got == 1.0).any() and (got == -1.0).any()


# ------------------------------------------------------------------ top layer
@pytest.mark.parametrize("c,m,h", [(10, 70, 1024), (2000, 70, 1024), (3307, 70, 1024), (3972, 70, 1024),
                                   (300, 1100, 1000), (129, 513, 33)])
def test_output_layer_bits_logp(B, torch_, real_path, c, m, h):
    rng = np.random.default_rng(c)
    hp = wl.make_bit_planes(m, h, 0.5, 31, B.packed_pitch(h))
    wout = rng.normal(0, 1 / np.sqrt(h), (c, h)).astype(np.float32)
    b = rng.normal(0, 0.1, c).astype(np.float32)
    prep = None
    if real_path != "fp32":
        prep = torch_.empty(B.bnn_output_prepared_bytes(c, h), dtype=torch_.uint8, device="cuda:0")
        B.bnn_output_prepare(dev(wout), prep)
    z = torch_.full((m, c + 1), 9.0, dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), z[:, :c], h, Hp=dev(hp), log_softmax=False, prepared=prep)
    zr = o.real_gemm_bits(hp, wout, b, h)
    assert np.abs(z.cpu().numpy()[:, :c] - zr).max() <= FLOAT_TOL * h
    lp = torch_.full((m, c + 1), 9.0, dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), lp[:, :c], h, Hp=dev(hp), prepared=prep)
    got = lp.cpu().numpy()
    assert np.abs(got[:, :c] - o.log_softmax(zr)).max() <= LOGP_TOL
    np.testing.assert_array_equal(got[:, c], 9.0)
    np.testing.assert_allclose(np.exp(got[:, :c].astype(np.float64)).sum(1), 1.0, atol=1e-4)


def test_output_layer_real_activations(B, torch_):
    m, h, c = 33, 300, 257
    rng = np.random.default_rng(8)
    hf = rng.uniform(-1, 1, (m, h)).astype(np.float32)
    wout = rng.normal(0, 1 / np.sqrt(h), (c, h)).astype(np.float32)
    b = rng.normal(0, 0.1, c).astype(np.float32)
    lp = torch_.empty((m, c), dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), lp, h, Hf=dev(hf))
    want = o.log_softmax(o.real_gemm_f32(hf, wout, b))
    assert np.abs(lp.cpu().numpy() - want).max() <= LOGP_TOL


@pytest.mark.parametrize("m,h,c", [(33, 300, 257), (600, 2048, 3400), (257, 33, 129), (1, 1, 1)])
def test_output_layer_real_activations_tensor_path(B, torch_, m, h, c):
    """fp32 activations x fp32 weights with both split into fp16 terms (bnn_output_layer_ws):
    the operand split costs at most 3 * 2^-22 * sum|a||w|; with the fp32 accumulation of 3 * H
    products on top the logits are tested at 2^-17 * sum|a||w|, the log-probs at 1e-4."""
    rng = np.random.default_rng(m + h + c)
    hf = rng.uniform(-1, 1, (m, h)).astype(np.float32)
    hf[rng.random(hf.shape) < 0.2] = 1.0          # hardtanh saturates often
    hf[rng.random(hf.shape) < 0.2] = -1.0
    hf[0, 0] = np.float32(1e-7)                   # below the fp16 normal range
    wout = rng.normal(0, 1 / np.sqrt(h), (c, h)).astype(np.float32)
    b = rng.normal(0, 0.1, c).astype(np.float32)
    prep = torch_.empty(B.bnn_output_prepared_bytes(c, h), dtype=torch_.uint8, device="cuda:0")
    B.bnn_output_prepare(dev(wout), prep)
    ws = torch_.empty(B.bnn_output_workspace_bytes(m, h), dtype=torch_.uint8, device="cuda:0")
    z = torch_.full((m, c + 1), 9.0, dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), z[:, :c], h, Hf=dev(hf), log_softmax=False, prepared=prep, workspace=ws)
    zr = o.real_gemm_f32(hf, wout, b)
    bound = 2.0 ** -17 * (np.abs(hf).astype(np.float64) @ np.abs(wout).astype(np.float64).T) + 1e-6
    got = z.cpu().numpy()
    assert (np.abs(got[:, :c] - zr) <= bound).all(), np.abs(got[:, :c] - zr).max()
    np.testing.assert_array_equal(got[:, c], 9.0)
    lp = torch_.empty((m, c), dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), dev(b), lp, h, Hf=dev(hf), prepared=prep, workspace=ws)
    assert np.abs(lp.cpu().numpy() - o.log_softmax(zr)).max() <= LOGP_TOL
    assert B.bnn_device_status() == 0


def test_output_layer_wide_dynamic_range_weights(B, torch_):
    """Rows whose magnitudes differ by many orders: the per-row power-of-two scaling of the
    prepared fp16 terms must keep every row accurate."""
    m, h, c = 64, 512, 200
    rng = np.random.default_rng(12)
    hp = wl.make_bit_planes(m, h, 0.5, 41, B.packed_pitch(h))
    wout = rng.normal(0, 1, (c, h)).astype(np.float32)
    wout *= (10.0 ** rng.uniform(-12, 6, (c, 1))).astype(np.float32)
    wout[5] = 0.0
    prep = torch_.empty(B.bnn_output_prepared_bytes(c, h), dtype=torch_.uint8, device="cuda:0")
    B.bnn_output_prepare(dev(wout), prep)
    z = torch_.empty((m, c), dtype=torch_.float32, device="cuda:0")
    B.bnn_output_layer(dev(wout), None, z, h, Hp=dev(hp), log_softmax=False, prepared=prep)
    zr = o.real_gemm_bits(hp, wout, None, h)
    bound = 2.0 ** -20 * np.abs(wout.astype(np.float64)).sum(1)[None, :]
    assert (np.abs(z.cpu().numpy() - zr) <= bound).all()
    assert B.bnn_device_status() == 0


@pytest.mark.parametrize("with_ws", [False, True])
@pytest.mark.parametrize("terms", [2, 3])
def test_signw_gemm_tensor_error_bound_by_terms(B, torch_, terms, with_ws):
    """2 bf16 terms: |err| <= 2^-16 sum|x|; 3 terms: products exact, only fp32 accumulation."""
    m, n, k = 300, 256, 440
    rng = np.random.default_rng(13)
    x = (rng.standard_normal((m, k)) * 10.0 ** rng.uniform(-3, 3, (m, 1))).astype(np.float32)
    wp = wl.make_bit_planes(n, k, 0.5, 42, B.packed_pitch(k))
    prev_p = B.bnn_set_option(B.OPT_REAL_PATH, B.PATH_TENSOR)
    prev_t = B.bnn_set_option(B.OPT_SIGNW_TERMS, terms)
    try:
        y = torch_.empty((m, n), dtype=torch_.float32, device="cuda:0")
        B.bnn_signw_gemm(dev(x), dev(wp), k, Y=y, workspace=signw_ws(B, "tensor_ws" if with_ws else "tensor", m, k))
        ref, sumabs = o.signw_gemm(x, wp, k)
        err = np.abs(y.cpu().numpy() - ref) / sumabs[:, None]
        assert err.max() <= (2.0 ** -16 if terms == 2 else 2.0 ** -21), err.max()
    finally:
        B.bnn_set_option(B.OPT_SIGNW_TERMS, prev_t)
        B.bnn_set_option(B.OPT_REAL_PATH, prev_p)
    assert B.bnn_device_status() == 0


# ------------------------------------------------------------------ pipe micro-benchmarks
def test_pipe_rate_launches_run_and_report_their_work(B, torch_):
    scratch = torch_.zeros(max(B.bnn_pipe_rate_scratch_bytes(k) for k in B.RATE_KINDS.values()), dtype=torch_.uint8,
                           device="cuda:0")
    for name, kind in B.RATE_KINDS.items():
        w1 = B.bnn_pipe_rate(kind, 1, scratch)
        w2 = B.bnn_pipe_rate(kind, 2, scratch)
        assert w1 > 0 and w2 == 2 * w1, name          # the work scales linearly with `repeat`
    torch_.cuda.synchronize()
    assert B.bnn_device_status() == 0
    with pytest.raises(B.BnnError):
        B.bnn_pipe_rate(99, 1, scratch)               # unknown kind
    with pytest.raises(B.BnnError):
        B.bnn_pipe_rate(0, 1, scratch[:1024])         # scratch too small


# ------------------------------------------------------------------ Sigmoid units (Table 2 topology)
@pytest.mark.parametrize("m,k,n", [(300, 440, 1024), (33, 77, 129), (700, 2048, 520)])
@pytest.mark.parametrize("tensor", [False, True])
def test_real_layer_sigmoid(B, torch_, m, k, n, tensor):
    """Real-valued weights x real input + bias, Sigmoid units (Eq. 1-2), FP32 pipe and tensor cores."""
    rng = np.random.default_rng(m + k + n)
    x = rng.standard_normal((m, k)).astype(np.float32)
    w = rng.normal(0, 1 / np.sqrt(k), (n, k)).astype(np.float32)
    b = rng.normal(0, 0.1, n).astype(np.float32)
    prep = ws = None
    if tensor:
        prep = torch_.empty(B.bnn_output_prepared_bytes(n, k), dtype=torch_.uint8, device="cuda:0")
        B.bnn_output_prepare(dev(w), prep)
        ws = torch_.empty(B.bnn_output_workspace_bytes(m, k), dtype=torch_.uint8, device="cuda:0")
    y = torch_.full((m, n + 2), 5.0, dtype=torch_.float32, device="cuda:0")
    B.bnn_real_layer(dev(x), dev(w), dev(b), y[:, :n], B.ACT_SIGMOID, prepared=prep, workspace=ws)
    _, want, _ = o.affine_act_f64(o.real_gemm_f32(x, w, b), None, None, o.ACT_SIGMOID)
    got = y.cpu().numpy()
    # |d sigmoid| <= |dz| / 4; the pre-activation is within 2^-17 sum|x||w| (tensor) or fp32 rounding
    bound = 0.25 * 2.0 ** -17 * (np.abs(x).astype(np.float64) @ np.abs(w).astype(np.float64).T) + 2e-7
    assert (np.abs(got[:, :n] - want) <= bound).all(), np.abs(got[:, :n] - want).max()
    np.testing.assert_array_equal(got[:, n:], 5.0)
    assert B.bnn_device_status() == 0


def test_affine_sigmoid_i32_in_place(B, torch_):
    rng = np.random.default_rng(77)
    m, n = 130, 200
    d = rng.integers(-2048, 2049, (m, n)).astype(np.int32)
    sc = rng.uniform(-0.01, 0.01, n).astype(np.float32)
    sh = rng.normal(0, 0.5, n).astype(np.float32)
    want = o.affine_sigmoid_i32(d, sc, sh)
    dd = dev(d)
    y = torch_.empty((m, n), dtype=torch_.float32, device="cuda:0")
    B.bnn_affine_sigmoid_i32(dd, dev(sc), dev(sh), y)
    assert np.abs(y.cpu().numpy() - want).max() <= 2e-7
    B.bnn_affine_sigmoid_i32(dd, dev(sc), dev(sh), dd.view(torch_.float32))     # same memory
    assert torch_.equal(dd.view(torch_.float32), y)
    B.bnn_affine_sigmoid_i32(dev(d), None, None, y)
    assert np.abs(y.cpu().numpy() - o.affine_sigmoid_i32(d, None, None)).max() <= 2e-7
