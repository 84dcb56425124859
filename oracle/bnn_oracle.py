"""ctypes front end of the plain-C CPU oracle (``bnn_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  Nothing in the CUDA package imports it, and it imports nothing from the
CUDA package.  All arrays are numpy host arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bnn_oracle.c")
_LIB = os.path.join(_HERE, "libbnn_oracle.so")

SIGN_ZERO_POS = 0
SIGN_ZERO_NEG = 1
ACT_NONE = 0
ACT_SIGN = 1
ACT_HARDTANH = 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
                               _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_sign_f32.argtypes = [C.c_float, C.c_int]
        _lib.oracle_sign_f32.restype = C.c_int
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _L(x):
    return C.c_long(int(x))


def words(k: int) -> int:
    return (k + 31) // 32


def sign(x: float, mode: int = SIGN_ZERO_POS) -> int:
    return int(lib().oracle_sign_f32(C.c_float(x), mode))


def sign_pack(X, mode=SIGN_ZERO_POS, pitch=None):
    X = _f32(X)
    M, K = X.shape
    ldp = words(K) if pitch is None else pitch
    P = np.empty((M, ldp), dtype=np.uint32)
    lib().oracle_sign_pack(_p(X), _L(M), _L(K), _L(K), _p(P), _L(ldp), C.c_int(mode))
    return P


def unpack_pm1(P, K):
    P = np.ascontiguousarray(P, dtype=np.uint32)
    M, ldp = P.shape
    S = np.empty((M, K), dtype=np.int8)
    lib().oracle_unpack_pm1(_p(P), _L(ldp), _L(M), _L(K), _p(S))
    return S


VALUES_PM1, VALUES_01 = 0, 1   # what the bits of a binary ACTIVATION stand for


def unpack_01(P, K):
    P = np.ascontiguousarray(P, dtype=np.uint32)
    M, ldp = P.shape
    S = np.empty((M, K), dtype=np.int8)
    lib().oracle_unpack_01(_p(P), _L(ldp), _L(M), _L(K), _p(S))
    return S


def gemm01(Hp, Wp, K):
    """d = sum_k h*w with h in {0,1} (bits of Hp) and w in {-1,+1} (bits of Wp)."""
    Hp = np.ascontiguousarray(Hp, dtype=np.uint32)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint32)
    M, N = Hp.shape[0], Wp.shape[0]
    D = np.empty((M, N), dtype=np.int32)
    lib().oracle_gemm01(_p(Hp), _L(Hp.shape[1]), _p(Wp), _L(Wp.shape[1]),
                        _L(M), _L(N), _L(K), _p(D), _L(N))
    return D


def xnor_gemm(Ap, Wp, K):
    Ap = np.ascontiguousarray(Ap, dtype=np.uint32)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint32)
    M, N = Ap.shape[0], Wp.shape[0]
    D = np.empty((M, N), dtype=np.int32)
    lib().oracle_xnor_gemm(_p(Ap), _L(Ap.shape[1]), _p(Wp), _L(Wp.shape[1]),
                           _L(M), _L(N), _L(K), _p(D), _L(N))
    return D


def affine_sign_pack_i32(D, scale, shift, mode=SIGN_ZERO_POS, pitch=None, want_y=False):
    D = np.ascontiguousarray(D, dtype=np.int32)
    M, N = D.shape
    scale, shift = _f32(scale), _f32(shift)
    ldp = words(N) if pitch is None else pitch
    P = np.empty((M, ldp), dtype=np.uint32)
    Y = np.empty((M, N), dtype=np.float32) if want_y else None
    lib().oracle_affine_sign_pack_i32(_p(D), _L(N), _L(M), _L(N), _p(scale), _p(shift),
                                      C.c_int(mode), _p(P), _L(ldp), _p(Y), _L(N))
    return (P, Y) if want_y else P


def signw_gemm(X, Wp, K):
    """Returns (Y float64 [M][N], sumabs float64 [M])."""
    X = _f32(X)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint32)
    M, N = X.shape[0], Wp.shape[0]
    assert X.shape[1] == K
    Y = np.empty((M, N), dtype=np.float64)
    sa = np.empty(M, dtype=np.float64)
    lib().oracle_signw_gemm(_p(X), _L(K), _p(Wp), _L(Wp.shape[1]), _L(M), _L(N), _L(K),
                            _p(Y), _L(N), _p(sa))
    return Y, sa


def affine_act_f64(Y, scale, shift, act, mode=SIGN_ZERO_POS, pitch=None):
    """Returns (Yhat f64, H f64, P uint32 or None)."""
    Y = np.ascontiguousarray(Y, dtype=np.float64)
    M, N = Y.shape
    scale, shift = _f32(scale), _f32(shift)
    Yh = np.empty((M, N), dtype=np.float64)
    H = np.empty((M, N), dtype=np.float64)
    P = None
    ldp = 0
    if act == ACT_SIGN:
        ldp = words(N) if pitch is None else pitch
        P = np.empty((M, ldp), dtype=np.uint32)
    lib().oracle_affine_act_f64(_p(Y), _L(N), _L(M), _L(N), _p(scale), _p(shift),
                                C.c_int(act), C.c_int(mode), _p(Yh), _L(N), _p(H), _L(N),
                                _p(P), _L(ldp))
    return Yh, H, P


def real_gemm_bits(Hp, Wout, b, H):
    Hp = np.ascontiguousarray(Hp, dtype=np.uint32)
    Wout, b = _f32(Wout), _f32(b)
    M, Cn = Hp.shape[0], Wout.shape[0]
    Z = np.empty((M, Cn), dtype=np.float64)
    lib().oracle_real_gemm_bits(_p(Hp), _L(Hp.shape[1]), _p(Wout), _L(Wout.shape[1]), _p(b),
                                _L(M), _L(Cn), _L(H), _p(Z), _L(Cn))
    return Z


def real_gemm_bits01(Hp, Wout, b, H):
    Hp = np.ascontiguousarray(Hp, dtype=np.uint32)
    Wout, b = _f32(Wout), _f32(b)
    M, Cn = Hp.shape[0], Wout.shape[0]
    Z = np.empty((M, Cn), dtype=np.float64)
    lib().oracle_real_gemm_bits01(_p(Hp), _L(Hp.shape[1]), _p(Wout), _L(Wout.shape[1]), _p(b),
                                  _L(M), _L(Cn), _L(H), _p(Z), _L(Cn))
    return Z


def real_gemm_f32(Hf, Wout, b):
    Hf, Wout, b = _f32(Hf), _f32(Wout), _f32(b)
    M, H = Hf.shape
    Cn = Wout.shape[0]
    Z = np.empty((M, Cn), dtype=np.float64)
    lib().oracle_real_gemm_f32(_p(Hf), _L(H), _p(Wout), _L(Wout.shape[1]), _p(b),
                               _L(M), _L(Cn), _L(H), _p(Z), _L(Cn))
    return Z


def log_softmax(Z):
    Z = np.ascontiguousarray(Z, dtype=np.float64)
    M, Cn = Z.shape
    LP = np.empty((M, Cn), dtype=np.float64)
    lib().oracle_log_softmax(_p(Z), _L(Cn), _L(M), _L(Cn), _p(LP), _L(Cn))
    return LP


ACT_SIGMOID = 3


def affine_sigmoid_i32(D, scale, shift):
    """h = Sigmoid(fma(scale, d, shift)) for integer dot products d; float64 [M][N]."""
    D = np.ascontiguousarray(D, dtype=np.int32)
    M, N = D.shape
    scale, shift = _f32(scale), _f32(shift)
    H = np.empty((M, N), dtype=np.float64)
    lib().oracle_affine_sigmoid_i32(_p(D), _L(N), _L(M), _L(N), _p(scale), _p(shift), _p(H), _L(N), None, _L(0))
    return H


def forward_mixed(X, W, scale, shift, Wout, bout, mode=SIGN_ZERO_POS, layer2_bits=None):
    """Forward pass of the paper's most accurate topology (Table 2, Section 3.2; with the binary
    weights of Section 2.3 in the middle): layer 1 keeps real-valued weights and Sigmoid units,
    layer 2 has +-1 weights on those real activations and Sign units, layers 3 .. L-1 are
    +-1 x +-1 with Sign units, layer L is +-1 x +-1 with Sigmoid units, the Softmax layer is
    real-valued.  W[0] is used as it is (bias shift[0], scale[0] must be None); W[1:] are
    binarised with Eq. 3.  ``layer2_bits`` replaces the oracle's own layer-2 bits (see forward).
    """
    X = _f32(X)
    L = len(W)
    assert L >= 3 and scale[0] is None
    taps = {"pre": [], "bits": []}
    Wp = [None] + [sign_pack(w, mode) for w in W[1:]]
    taps["Wp"] = Wp
    # layer 1: real weights, Sigmoid (Eq. 1-2 with f = Sigmoid), in double, handed on as fp32
    Y1 = real_gemm_f32(X, W[0], shift[0])
    _, H1, _ = affine_act_f64(Y1, None, None, ACT_SIGMOID, mode)
    taps["h1"] = H1
    h1 = H1.astype(np.float32)
    # layer 2: +-1 weights on real activations, Sign
    Y2, sumabs = signw_gemm(h1, Wp[1], W[1].shape[1])
    Yh, _, P = affine_act_f64(Y2, scale[1], shift[1], ACT_SIGN, mode)
    taps["sumabs2"], taps["pre2"], taps["bits_own_layer2"] = sumabs, Yh, P
    if layer2_bits is not None:
        P = np.ascontiguousarray(layer2_bits, dtype=np.uint32)[:, :words(W[1].shape[0])]
    taps["bits"].append(P)
    for l in range(2, L - 1):
        D = xnor_gemm(P, Wp[l], W[l].shape[1])
        P = affine_sign_pack_i32(D, scale[l], shift[l], mode)
        taps["bits"].append(P)
    # layer L: +-1 x +-1, Sigmoid units
    D = xnor_gemm(P, Wp[L - 1], W[L - 1].shape[1])
    HL = affine_sigmoid_i32(D, scale[L - 1], shift[L - 1])
    taps["hL"] = HL
    Z = real_gemm_f32(HL.astype(np.float32), Wout, bout)
    taps["logits"] = Z
    taps["logp"] = log_softmax(Z)
    return taps


def splice(F, left, right):
    """Context window of the feature front end (Section 3: frames spliced over a context of 11):
    row m of the result is the concatenation of rows m - left .. m + right of F; rows outside the
    matrix are replaced by the nearest existing one (the paper does not say how edges are padded;
    this is the reading taken).  Written out as plain loops."""
    F = _f32(F)
    M, D = F.shape
    out = np.empty((M, (left + right + 1) * D), dtype=np.float32)
    for m in range(M):
        for j, t in enumerate(range(-left, right + 1)):
            r = min(max(m + t, 0), M - 1)
            out[m, j * D:(j + 1) * D] = F[r]
    return out


def forward(X, W, scale, shift, Wout, bout, act=ACT_SIGN, mode=SIGN_ZERO_POS,
            layer1_bits=None, values=VALUES_PM1, log_prior=None):
    """Whole forward pass, layer by layer in the order of Algorithms 1 and 2.

    W: list of real-valued weight matrices [N_l][K_l]; they are binarised with Eq. 3 first.
    act == ACT_SIGN: layer 1 is +-1 weights on real input, later hidden layers are +-1 x +-1;
    act == ACT_HARDTANH: every hidden layer is +-1 weights on real activations.
    ``layer1_bits`` (optional) replaces the oracle's own first-layer bits, so that a caller
    can continue from another implementation's decision on values inside the float
    tolerance band.  ``values`` = VALUES_01 makes the binary activations (0,1) instead of
    (-1,+1) (Section 3.2): the stored bit is the same decision (pre-activation above / at zero),
    it stands for 1 / 0 in the layer that consumes it.  Returns a dict of per-layer taps and ``logp``.
    """
    X = _f32(X)
    taps = {"Wp": [], "pre": [], "bits": [], "h": []}
    Wp = [sign_pack(w, mode) for w in W]
    taps["Wp"] = Wp
    K = X.shape[1]
    if act == ACT_SIGN:
        Y, sumabs = signw_gemm(X, Wp[0], K)
        Yh, _, P = affine_act_f64(Y, scale[0], shift[0], ACT_SIGN, mode)
        taps["sumabs"] = sumabs
        taps["pre"].append(Yh)
        taps["bits_own_layer1"] = P
        if layer1_bits is not None:
            P = np.ascontiguousarray(layer1_bits, dtype=np.uint32)[:, :words(W[0].shape[0])]
        taps["bits"].append(P)
        for l in range(1, len(W)):
            D = (gemm01 if values == VALUES_01 else xnor_gemm)(P, Wp[l], W[l].shape[1])
            P = affine_sign_pack_i32(D, scale[l], shift[l], mode)
            taps["pre"].append(D)
            taps["bits"].append(P)
        Z = (real_gemm_bits01 if values == VALUES_01 else real_gemm_bits)(P, Wout, bout, Wout.shape[1])
    else:
        Hf = X
        for l in range(len(W)):
            Y, sumabs = signw_gemm(Hf, Wp[l], W[l].shape[1])
            Yh, Hd, _ = affine_act_f64(Y, scale[l], shift[l], act, mode)
            taps["pre"].append(Yh)
            taps["h"].append(Hd)
            taps.setdefault("sumabs_l", []).append(sumabs)
            Hf = Hd.astype(np.float32)
        Z = real_gemm_f32(Hf, Wout, bout)
    taps["logits"] = Z
    taps["logp"] = log_softmax(Z)
    if log_prior is not None:   # scaled log-likelihoods for a hybrid decoder: log p(s|x) - log p(s)
        taps["logp"] = taps["logp"] - np.asarray(log_prior, dtype=np.float64)[None, :]
    return taps
