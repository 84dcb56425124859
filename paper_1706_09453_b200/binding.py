"""Thin ctypes binding of the C ABI in ``include/bnn.h``.

Argument marshalling only: every function takes torch CUDA tensors (device memory) and the
current torch stream, calls the entry point of the same name and raises on a non-zero
status.  There is no CPU path; a missing library or a CPU tensor is an error.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

SIGN_ZERO_POS, SIGN_ZERO_NEG = 0, 1
ACT_NONE, ACT_SIGN_PACK, ACT_HARDTANH, ACT_SIGMOID = 0, 1, 2, 3
VALUES_PM1, VALUES_01 = 0, 1
LAYER_SIGNW, LAYER_XNOR, LAYER_REAL_OUT, LAYER_REAL = 0, 1, 2, 3


class BnnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class Epilogue(C.Structure):
    _fields_ = [("act", C.c_int), ("sign_mode", C.c_int),
                ("scale", C.c_void_p), ("shift", C.c_void_p),
                ("thr", C.c_void_p), ("flip", C.c_void_p),
                ("out_bits", C.c_void_p), ("ldob", C.c_int)]


class Layer(C.Structure):
    _fields_ = [("kind", C.c_int), ("K", C.c_int), ("N", C.c_int),
                ("Wp", C.c_void_p), ("ldwp", C.c_int),
                ("W", C.c_void_p), ("ldw", C.c_int), ("W_prepared", C.c_void_p),
                ("scale", C.c_void_p), ("shift", C.c_void_p),
                ("thr", C.c_void_p), ("flip", C.c_void_p),
                ("act", C.c_int)]


class Model(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("sign_mode", C.c_int), ("layers", C.POINTER(Layer)),
                ("act_values", C.c_int), ("splice_left", C.c_int), ("splice_right", C.c_int),
                ("log_prior", C.c_void_p)]


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Load the CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            raise ImportError("CUDA library %s is missing: run paper_1706_09453_b200.build.build() "
                              "(there is no CPU fallback)" % path)
        L = C.CDLL(path)
        L.bnn_status_string.restype = C.c_char_p
        L.bnn_status_string.argtypes = [C.c_int]
        L.bnn_packed_pitch.restype = C.c_int
        L.bnn_packed_pitch.argtypes = [C.c_int]
        L.bnn_set_option.argtypes = [C.c_int, C.c_int]
        L.bnn_set_option.restype = C.c_int
        L.bnn_output_prepared_bytes.argtypes = [C.c_int, C.c_int]
        L.bnn_output_prepared_bytes.restype = C.c_size_t
        L.bnn_output_prepare.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.bnn_output_prepare.restype = C.c_int
        L.bnn_xnor_prepared_bytes.argtypes = [C.c_int, C.c_int]
        L.bnn_xnor_prepared_bytes.restype = C.c_size_t
        L.bnn_xnor_prepare.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
        L.bnn_xnor_prepare.restype = C.c_int
        L.bnn_xnor_gemm_prepared.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                             C.c_int, C.POINTER(Epilogue), C.c_void_p]
        L.bnn_xnor_gemm_prepared.restype = C.c_int
        L.bnn_pipe_rate_scratch_bytes.argtypes = [C.c_int]
        L.bnn_pipe_rate_scratch_bytes.restype = C.c_size_t
        L.bnn_pipe_rate.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.POINTER(C.c_double), C.c_void_p]
        L.bnn_pipe_rate.restype = C.c_int
        L.bnn_device_status.argtypes = [C.POINTER(C.c_int)]
        L.bnn_device_status.restype = C.c_int
        L.bnn_query_status.argtypes = [C.c_void_p, C.c_void_p]
        L.bnn_query_status.restype = C.c_int
        L.bnn_reset_status.argtypes = [C.c_void_p]
        L.bnn_reset_status.restype = C.c_int
        L.bnn_wait_probe.argtypes = [C.c_void_p]
        L.bnn_wait_probe.restype = C.c_int
        L.bnn_forward_workspace_bytes.restype = C.c_size_t
        L.bnn_forward_workspace_bytes.argtypes = [C.POINTER(Model), C.c_int]
        L.bnn_forward_min_workspace_bytes.restype = C.c_size_t
        L.bnn_forward_min_workspace_bytes.argtypes = [C.POINTER(Model), C.c_int]
        L.bnn_signw_workspace_bytes.restype = C.c_size_t
        L.bnn_signw_workspace_bytes.argtypes = [C.c_int, C.c_int]
        L.bnn_signw_gemm_ws.restype = C.c_int
        L.bnn_signw_gemm_ws.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                        C.c_int, C.POINTER(Epilogue), C.c_void_p, C.c_size_t, C.c_void_p]
        i, p = C.c_int, C.c_void_p
        L.bnn_pack_weights.argtypes = [p, i, i, i, p, i, i, p]
        L.bnn_binarize_pack.argtypes = [p, i, i, i, p, i, i, p]
        L.bnn_fold_thresholds.argtypes = [p, p, i, i, i, p, p, p]
        L.bnn_xnor_gemm.argtypes = [p, i, p, i, i, i, i, p, i, C.POINTER(Epilogue), p]
        L.bnn_signw_gemm.argtypes = [p, i, p, i, i, i, i, p, i, C.POINTER(Epilogue), p]
        L.bnn_output_layer.argtypes = [p, i, p, i, p, i, p, p, i, i, i, p, i, i, p]
        L.bnn_output_layer01.argtypes = [p, i, p, i, p, p, i, i, i, p, i, i, p]
        L.bnn_output_layer01.restype = C.c_int
        L.bnn_output_workspace_bytes.argtypes = [i, i]
        L.bnn_output_workspace_bytes.restype = C.c_size_t
        L.bnn_output_layer_ws.argtypes = [p, i, p, i, p, p, i, i, i, p, i, i, p, C.c_size_t, p]
        L.bnn_output_layer_ws.restype = C.c_int
        L.bnn_real_layer.argtypes = [p, i, p, i, p, p, i, i, i, p, i, i, p, C.c_size_t, p]
        L.bnn_real_layer.restype = C.c_int
        L.bnn_affine_sigmoid_i32.argtypes = [p, i, p, p, i, i, p, i, p]
        L.bnn_affine_sigmoid_i32.restype = C.c_int
        L.bnn_gemm01.argtypes = [p, i, p, i, p, i, i, i, p, i, C.POINTER(Epilogue), p]
        L.bnn_gemm01.restype = C.c_int
        L.bnn_forward.argtypes = [C.POINTER(Model), p, i, i, p, i, p, C.c_size_t, C.POINTER(p), p]
        L.bnn_forward_static.argtypes = [C.POINTER(Model), p, i, i, p, i, p]
        L.bnn_forward_static.restype = C.c_int
        L.bnn_forward_events.argtypes = [C.POINTER(Model), p, i, i, p, i, p, C.c_size_t, C.POINTER(p),
                                         C.POINTER(p), p]
        for name in ("bnn_pack_weights", "bnn_binarize_pack", "bnn_fold_thresholds", "bnn_xnor_gemm",
                     "bnn_signw_gemm", "bnn_output_layer", "bnn_forward", "bnn_forward_events"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().bnn_status_string(int(status)).decode()


def packed_pitch(k: int) -> int:
    return int(lib().bnn_packed_pitch(int(k)))


OPT_XNOR_PATH, OPT_REAL_PATH, OPT_SIGNW_TERMS, OPT_XNOR_PREPARED, OPT_SMALL_BATCH, OPT_XNOR_STACK, OPT_WAIT_LIMIT_US = 0, 1, 2, 3, 4, 5, 6
OPT_SOFTMAX_FOLLOW = 7
ERR_TIMEOUT = 7
PREPARED_AUTO, PREPARED_STREAM, PREPARED_RESIDENT = 0, 1, 2
PATH_AUTO, PATH_CUDA_CORE, PATH_TENSOR = 0, 1, 2
XNOR_AUTO, XNOR_POPC, XNOR_TENSOR = PATH_AUTO, PATH_CUDA_CORE, PATH_TENSOR


def bnn_set_option(option: int, value: int) -> int:
    prev = int(lib().bnn_set_option(int(option), int(value)))
    if prev < 0:
        raise ValueError("unknown option/value %r/%r" % (option, value))
    return prev


def bnn_set_xnor_path(path: int) -> int:
    return bnn_set_option(OPT_XNOR_PATH, path)


RATE_KINDS = {"popc": 0, "lop3": 1, "iadd": 2, "fadd": 3, "ffma": 4, "mma_mxf4_n256": 5, "mma_mxf4_n192": 6,
              "mma_mxf4_n192_atmem": 7, "mma_f16_n256": 8, "l2_read": 9}


def bnn_pipe_rate_scratch_bytes(which: int) -> int:
    return lib().bnn_pipe_rate_scratch_bytes(which)


def bnn_pipe_rate(which: int, repeat: int, scratch) -> float:
    """Enqueues one micro-benchmark launch on the current stream; returns the work it performs."""
    work = C.c_double(0.0)
    _check(lib().bnn_pipe_rate(which, repeat, _ptr(scratch), scratch.numel() * scratch.element_size(),
                               C.byref(work), _stream()), "bnn_pipe_rate")
    return work.value


def bnn_device_status() -> int:
    """Synchronises the device; 0 unless a tensor-core kernel gave up on a bounded wait."""
    st = C.c_int(-1)
    rc = lib().bnn_device_status(C.byref(st))
    if rc not in (0, ERR_TIMEOUT):
        _check(rc, "bnn_device_status")
    return st.value


def bnn_query_status(dst):
    """Enqueues a copy of the status word into ``dst`` (int32 CUDA or pinned tensor) on the current stream."""
    _check(lib().bnn_query_status(C.c_void_p(dst.data_ptr()), _stream()), "bnn_query_status")


def bnn_reset_status():
    _check(lib().bnn_reset_status(_stream()), "bnn_reset_status")


def bnn_wait_probe():
    """Enqueues the launch whose wait runs out (sets the status word after the wait limit)."""
    _check(lib().bnn_wait_probe(_stream()), "bnn_wait_probe")


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("expected a CUDA tensor (there is no CPU path)")
    if dtype is not None and t.dtype != dtype:
        raise TypeError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def _ld(t):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with contiguous rows")
    return t.stride(0)


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(rc, where):
    if rc != 0:
        raise BnnError(rc, where)


def raw_call(name, *args) -> int:
    """Call an entry point with raw integers/pointers and return its status (for tests)."""
    return int(getattr(lib(), name)(*args))


def bnn_pack_weights(W, Wp, sign_mode=SIGN_ZERO_POS):
    n, k = W.shape
    _check(lib().bnn_pack_weights(_ptr(W, torch.float32), n, k, _ld(W), _ptr(Wp, torch.int32), _ld(Wp),
                                  sign_mode, _stream()), "bnn_pack_weights")
    return Wp


def bnn_binarize_pack(X, Ap, sign_mode=SIGN_ZERO_POS):
    m, k = X.shape
    _check(lib().bnn_binarize_pack(_ptr(X, torch.float32), m, k, _ld(X), _ptr(Ap, torch.int32), _ld(Ap),
                                   sign_mode, _stream()), "bnn_binarize_pack")
    return Ap


def bnn_fold_thresholds(scale, shift, N, K, thr, flip, sign_mode=SIGN_ZERO_POS):
    _check(lib().bnn_fold_thresholds(_ptr(scale, torch.float32), _ptr(shift, torch.float32), N, K, sign_mode,
                                     _ptr(thr, torch.int32), _ptr(flip, torch.int32), _stream()),
           "bnn_fold_thresholds")
    return thr, flip


def _epilogue(act=ACT_NONE, sign_mode=SIGN_ZERO_POS, scale=None, shift=None, thr=None, flip=None,
              out_bits=None):
    e = Epilogue()
    e.act, e.sign_mode = act, sign_mode
    e.scale, e.shift = _ptr(scale, torch.float32), _ptr(shift, torch.float32)
    e.thr, e.flip = _ptr(thr, torch.int32), _ptr(flip, torch.int32)
    e.out_bits = _ptr(out_bits, torch.int32)
    e.ldob = _ld(out_bits) if out_bits is not None else 0
    return e


def bnn_xnor_gemm(Ap, Wp, K, C_out=None, thr=None, flip=None, out_bits=None):
    """Packed tensors are int32 views of the uint32 words ([rows][pitch])."""
    m, n = Ap.shape[0], Wp.shape[0]
    e = None
    if out_bits is not None:
        e = C.byref(_epilogue(ACT_SIGN_PACK, thr=thr, flip=flip, out_bits=out_bits))
    _check(lib().bnn_xnor_gemm(_ptr(Ap, torch.int32), _ld(Ap), _ptr(Wp, torch.int32), _ld(Wp), m, n, K,
                               _ptr(C_out, torch.int32), _ld(C_out) if C_out is not None else 0,
                               e, _stream()), "bnn_xnor_gemm")


def bnn_xnor_prepared_bytes(N, K) -> int:
    return int(lib().bnn_xnor_prepared_bytes(int(N), int(K)))


def bnn_xnor_prepare(Wp, K, prepared):
    """Packed weights [N][pitch] -> their widened image in ``prepared`` (uint8 CUDA tensor)."""
    _check(lib().bnn_xnor_prepare(_ptr(Wp, torch.int32), _ld(Wp), Wp.shape[0], K, _ptr(prepared),
                                  prepared.numel() * prepared.element_size(), _stream()), "bnn_xnor_prepare")
    return prepared


def bnn_xnor_gemm_prepared(Ap, prepared, N, K, C_out=None, thr=None, flip=None, out_bits=None):
    """bnn_xnor_gemm with the weights given as the image bnn_xnor_prepare made of them."""
    e = None
    if out_bits is not None:
        e = C.byref(_epilogue(ACT_SIGN_PACK, thr=thr, flip=flip, out_bits=out_bits))
    _check(lib().bnn_xnor_gemm_prepared(_ptr(Ap, torch.int32), _ld(Ap), _ptr(prepared), Ap.shape[0], N, K,
                                        _ptr(C_out, torch.int32), _ld(C_out) if C_out is not None else 0,
                                        e, _stream()), "bnn_xnor_gemm_prepared")


def bnn_gemm01(Hp, Wp, K, N=None, prepared=None, C_out=None, thr=None, flip=None, out_bits=None):
    """Activations in (0,1) x weights in (-1,+1); ``Wp`` and/or ``prepared`` give the weights."""
    n = Wp.shape[0] if Wp is not None else N
    e = None
    if out_bits is not None:
        e = C.byref(_epilogue(ACT_SIGN_PACK, thr=thr, flip=flip, out_bits=out_bits))
    _check(lib().bnn_gemm01(_ptr(Hp, torch.int32), _ld(Hp), _ptr(Wp, torch.int32), _ld(Wp) if Wp is not None else 0,
                            _ptr(prepared), Hp.shape[0], n, K,
                            _ptr(C_out, torch.int32), _ld(C_out) if C_out is not None else 0,
                            e, _stream()), "bnn_gemm01")


def bnn_signw_workspace_bytes(M, K) -> int:
    return int(lib().bnn_signw_workspace_bytes(int(M), int(K)))


def bnn_signw_gemm(X, Wp, K, Y=None, act=ACT_NONE, scale=None, shift=None, out_bits=None,
                   sign_mode=SIGN_ZERO_POS, workspace=None):
    """With ``workspace`` (uint8 CUDA tensor) this calls bnn_signw_gemm_ws."""
    m, n = X.shape[0], Wp.shape[0]
    e = C.byref(_epilogue(act, sign_mode, scale, shift, out_bits=out_bits))
    if workspace is not None:
        _check(lib().bnn_signw_gemm_ws(_ptr(X, torch.float32), _ld(X), _ptr(Wp, torch.int32), _ld(Wp), m, n, K,
                                       _ptr(Y, torch.float32), _ld(Y) if Y is not None else 0, e,
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
               "bnn_signw_gemm_ws")
        return
    _check(lib().bnn_signw_gemm(_ptr(X, torch.float32), _ld(X), _ptr(Wp, torch.int32), _ld(Wp), m, n, K,
                                _ptr(Y, torch.float32), _ld(Y) if Y is not None else 0, e, _stream()),
           "bnn_signw_gemm")


def bnn_output_prepared_bytes(C_, H) -> int:
    return int(lib().bnn_output_prepared_bytes(int(C_), int(H)))


def bnn_output_prepare(Wout, prepared):
    c, h = Wout.shape
    _check(lib().bnn_output_prepare(_ptr(Wout, torch.float32), _ld(Wout), c, h, _ptr(prepared),
                                    prepared.numel() * prepared.element_size(), _stream()), "bnn_output_prepare")
    return prepared


def bnn_real_layer(Hf, W, bias, Y, act=ACT_SIGMOID, prepared=None, workspace=None):
    """Y = act(Hf W^T + bias) with real-valued weights; tensor cores with ``prepared`` and ``workspace``."""
    m, k = Hf.shape
    _check(lib().bnn_real_layer(_ptr(Hf, torch.float32), _ld(Hf), _ptr(W, torch.float32), _ld(W),
                                _ptr(bias, torch.float32), _ptr(prepared), m, W.shape[0], k,
                                _ptr(Y, torch.float32), _ld(Y), act, _ptr(workspace),
                                workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                _stream()), "bnn_real_layer")
    return Y


def bnn_affine_sigmoid_i32(D, scale, shift, Y):
    """Y = Sigmoid(fma(scale, D, shift)); ``Y`` may be a float32 view of ``D``'s own memory."""
    m, n = D.shape
    _check(lib().bnn_affine_sigmoid_i32(_ptr(D, torch.int32), _ld(D), _ptr(scale, torch.float32),
                                        _ptr(shift, torch.float32), m, n, _ptr(Y, torch.float32), _ld(Y),
                                        _stream()), "bnn_affine_sigmoid_i32")
    return Y


def bnn_output_workspace_bytes(M, H) -> int:
    return int(lib().bnn_output_workspace_bytes(int(M), int(H)))


def bnn_output_layer(Wout, b, logp, H, Hp=None, Hf=None, log_softmax=True, prepared=None, values=VALUES_PM1,
                     workspace=None):
    """``workspace`` (uint8 CUDA tensor) with fp32 activations ``Hf`` calls bnn_output_layer_ws."""
    m = (Hp if Hp is not None else Hf).shape[0]
    c = Wout.shape[0]
    if workspace is not None:
        _check(lib().bnn_output_layer_ws(_ptr(Hf, torch.float32), _ld(Hf), _ptr(Wout, torch.float32), _ld(Wout),
                                         _ptr(b, torch.float32), _ptr(prepared), m, c, H,
                                         _ptr(logp, torch.float32), _ld(logp), int(log_softmax),
                                         _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
               "bnn_output_layer_ws")
        return logp
    if values == VALUES_01:
        _check(lib().bnn_output_layer01(_ptr(Hp, torch.int32), _ld(Hp), _ptr(Wout, torch.float32), _ld(Wout),
                                        _ptr(b, torch.float32), _ptr(prepared), m, c, H,
                                        _ptr(logp, torch.float32), _ld(logp), int(log_softmax), _stream()),
               "bnn_output_layer01")
        return logp
    _check(lib().bnn_output_layer(_ptr(Hp, torch.int32), _ld(Hp) if Hp is not None else 0,
                                  _ptr(Hf, torch.float32), _ld(Hf) if Hf is not None else 0,
                                  _ptr(Wout, torch.float32), _ld(Wout), _ptr(b, torch.float32),
                                  _ptr(prepared), m, c, H, _ptr(logp, torch.float32), _ld(logp), int(log_softmax), _stream()),
           "bnn_output_layer")
    return logp


class ModelDesc:
    """Host-side bnn_model built from a list of layer dicts; keeps the tensors alive."""

    def __init__(self, layers, sign_mode=SIGN_ZERO_POS, act_values=VALUES_PM1, splice=(0, 0), log_prior=None):
        self._keep = (layers, log_prior)
        arr = (Layer * len(layers))()
        for a, d in zip(arr, layers):
            a.kind, a.K, a.N, a.act = d["kind"], d["K"], d["N"], d.get("act", ACT_NONE)
            wp, w = d.get("Wp"), d.get("W")
            a.Wp, a.ldwp = _ptr(wp, torch.int32), (_ld(wp) if wp is not None else 0)
            a.W, a.ldw = _ptr(w, torch.float32), (_ld(w) if w is not None else 0)
            a.W_prepared = _ptr(d.get("W_prepared"))
            a.scale, a.shift = _ptr(d.get("scale"), torch.float32), _ptr(d.get("shift"), torch.float32)
            a.thr, a.flip = _ptr(d.get("thr"), torch.int32), _ptr(d.get("flip"), torch.int32)
        self._arr = arr
        self.c = Model(len(layers), sign_mode, arr, act_values, splice[0], splice[1], _ptr(log_prior, torch.float32))
        self.layers = layers

    def workspace_bytes(self, M: int) -> int:
        return int(lib().bnn_forward_workspace_bytes(C.byref(self.c), M))

    def min_workspace_bytes(self, M: int) -> int:
        return int(lib().bnn_forward_min_workspace_bytes(C.byref(self.c), M))


def bnn_forward(model: ModelDesc, X, logp, workspace, layer_out=None):
    m = X.shape[0]
    lo = None
    if layer_out is not None:
        lo = (C.c_void_p * len(layer_out))(*[(_ptr(t) if t is not None else None) for t in layer_out])
    _check(lib().bnn_forward(C.byref(model.c), _ptr(X, torch.float32), _ld(X), m,
                             _ptr(logp, torch.float32), _ld(logp),
                             _ptr(workspace), workspace.numel() * workspace.element_size(),
                             lo, _stream()), "bnn_forward")
    return logp


def bnn_forward_events(model: ModelDesc, X, logp, workspace, events, layer_out=None):
    """``events``: n_layers+2 recorded-at-least-once torch.cuda.Event objects (timing enabled)."""
    m = X.shape[0]
    lo = None
    if layer_out is not None:
        lo = (C.c_void_p * len(layer_out))(*[(_ptr(t) if t is not None else None) for t in layer_out])
    ev = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
    _check(lib().bnn_forward_events(C.byref(model.c), _ptr(X, torch.float32), _ld(X), m,
                                    _ptr(logp, torch.float32), _ld(logp),
                                    _ptr(workspace), workspace.numel() * workspace.element_size(),
                                    lo, ev, _stream()), "bnn_forward_events")
    return logp


STATIC_WORKSPACE_BYTES = 8 << 20


def bnn_forward_static(model: ModelDesc, X, logp):
    """Forward pass that allocates nothing: its scratch is a fixed array inside the library
    (for callers that may not call cudaMalloc).  Raises BnnError(status 5) when the batch
    needs more than STATIC_WORKSPACE_BYTES of scratch."""
    _check(lib().bnn_forward_static(C.byref(model.c), _ptr(X, torch.float32), _ld(X), X.shape[0],
                                    _ptr(logp, torch.float32), _ld(logp), _stream()), "bnn_forward_static")
    return logp
