"""Host-side checks of the C ABI that need no GPU: the library loads, exports every function
the header declares, and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1706_09453_b200 import build, binding
    build.build()
    return binding.lib()


def declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"BNN_API\s+[\w\s\*]+?\b(bnn_\w+)\s*\(", src)
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"bnn_pack_weights", "bnn_binarize_pack", "bnn_xnor_gemm", "bnn_signw_gemm",
            "bnn_forward"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None, n


def test_status_strings_and_pitch(lib):
    from paper_1706_09453_b200 import binding as B
    assert B.status_string(0) == "ok"
    assert len({B.status_string(i) for i in range(8)}) == 8
    assert [B.packed_pitch(k) for k in (1, 32, 33, 128, 129, 440, 2048)] == [4, 4, 4, 4, 8, 16, 64]


def test_bad_arguments_are_rejected_without_a_launch(lib):
    from paper_1706_09453_b200 import binding as B
    fake = 0x10000  # 16-byte aligned non-NULL "pointer": never dereferenced on the host
    rc = B.raw_call
    # NULL pointers
    assert rc("bnn_pack_weights", None, 4, 4, 4, fake, 4, 0, None) == 1
    assert rc("bnn_binarize_pack", fake, 4, 4, 4, None, 4, 0, None) == 1
    # sizes and pitches
    assert rc("bnn_pack_weights", fake, 0, 4, 4, fake, 4, 0, None) == 2
    assert rc("bnn_pack_weights", fake, 4, 8, 4, fake, 4, 0, None) == 2      # ldw < K
    assert rc("bnn_pack_weights", fake, 4, 200, 200, fake, 4, 0, None) == 2  # pitch < ceil(K/32)
    # alignment
    assert rc("bnn_pack_weights", fake, 4, 4, 4, fake, 6, 0, None) == 3
    assert rc("bnn_pack_weights", fake, 4, 4, 4, fake + 4, 4, 0, None) == 3
    # sign mode
    assert rc("bnn_pack_weights", fake, 4, 4, 4, fake, 4, 7, None) == 4
    # xnor: K too large, neither C nor epilogue, bad epilogue
    assert rc("bnn_xnor_gemm", fake, 4, fake, 4, 1, 1, (1 << 24) + 1, fake, 1, None, None) == 2
    assert rc("bnn_xnor_gemm", fake, 4, fake, 4, 1, 1, 32, None, 0, None, None) == 1
    e = B.Epilogue()
    e.act = B.ACT_HARDTANH
    assert rc("bnn_xnor_gemm", fake, 4, fake, 4, 1, 1, 32, fake, 1, C.byref(e), None) == 4
    e.act = B.ACT_SIGN_PACK
    assert rc("bnn_xnor_gemm", fake, 4, fake, 4, 1, 1, 32, fake, 1, C.byref(e), None) == 1  # thr NULL
    assert rc("bnn_xnor_gemm", fake, 4, fake, 4, 1, 40, 32, fake, 8, None, None) == 2       # ldc < N
    # signw / output layer
    assert rc("bnn_signw_gemm", None, 4, fake, 4, 1, 1, 4, fake, 1, None, None) == 1
    assert rc("bnn_signw_gemm", fake, 4, fake, 4, 1, 1, 4, None, 0, None, None) == 1        # no output
    assert rc("bnn_output_layer", fake, 4, fake, 4, fake, 4, None, None, 1, 1, 4, fake, 1, 1, None) == 4
    assert rc("bnn_output_layer", None, 0, None, 0, fake, 4, None, None, 1, 1, 4, fake, 1, 1, None) == 1
    assert rc("bnn_output_layer", fake, 4, None, 0, fake, 4, None, fake + 16, 1, 1, 4, fake, 1, 1, None) == 3
    assert rc("bnn_output_prepare", fake, 4, 1, 4, None, 1 << 20, None) == 1
    assert rc("bnn_output_prepare", fake, 4, 1, 4, fake, 16, None) == 5
    assert B.bnn_output_prepared_bytes(3400, 2048) == 27 * 64 * 16384 + 27 * 128 * 4
    # prepared weights of a binary layer
    assert B.bnn_xnor_prepared_bytes(2048, 2048) == 8 * 2304 * 128
    assert B.bnn_xnor_prepared_bytes(1, 1) == 384 * 128
    assert B.bnn_xnor_prepared_bytes(4, (1 << 22) + 1) == 0
    assert rc("bnn_xnor_prepare", fake, 4, 4, 32, None, 1 << 20, None) == 1
    assert rc("bnn_xnor_prepare", None, 4, 4, 32, fake, 1 << 20, None) == 1
    assert rc("bnn_xnor_prepare", fake, 4, 0, 32, fake, 1 << 20, None) == 2
    assert rc("bnn_xnor_prepare", fake, 4, 4, 32, fake, 100, None) == 5
    assert rc("bnn_xnor_prepare", fake, 4, 4, 32, fake + 16, 1 << 20, None) == 3
    assert rc("bnn_xnor_prepare", fake, 1 << 18, 4, (1 << 22) + 1, fake, 1 << 30, None) == 4
    assert rc("bnn_xnor_gemm_prepared", fake, 4, None, 1, 1, 32, fake, 1, None, None) == 1
    assert rc("bnn_xnor_gemm_prepared", fake, 4, fake + 16, 1, 1, 32, fake, 1, None, None) == 3
    assert rc("bnn_xnor_gemm_prepared", fake, 4, fake, 1, 1, 32, None, 0, None, None) == 1
    assert rc("bnn_xnor_gemm_prepared", fake, 4, fake, 1, 40, 32, fake, 8, None, None) == 2
    # top layer with scratch
    assert B.bnn_output_workspace_bytes(8192, 2048) == 32 * 64 * 32768
    assert rc("bnn_output_layer_ws", None, 4, fake, 4, None, None, 1, 1, 4, fake, 1, 1, None, 0, None) == 1
    assert rc("bnn_output_layer_ws", fake, 2, fake, 4, None, None, 1, 1, 4, fake, 1, 1, None, 0, None) == 2
    # (0,1) activations
    assert rc("bnn_gemm01", fake, 4, None, 0, None, 1, 1, 32, fake, 1, None, None) == 1     # no weights at all
    assert rc("bnn_gemm01", fake, 4, fake, 4, None, 1, 1, 32, None, 0, None, None) == 1     # no output
    assert rc("bnn_gemm01", fake, 4, fake, 6, None, 1, 1, 32, fake, 1, None, None) == 3     # weight pitch
    assert rc("bnn_gemm01", fake, 4, None, 0, fake + 16, 1, 1, 32, fake, 1, None, None) == 3
    assert rc("bnn_output_layer01", None, 4, fake, 4, None, None, 1, 1, 4, fake, 1, 1, None) == 1
    assert rc("bnn_output_layer01", fake, 4, fake, 2, None, None, 1, 1, 4, fake, 1, 1, None) == 2
    # options
    assert B.bnn_set_option(B.OPT_XNOR_PATH, B.PATH_CUDA_CORE) == 0
    assert B.bnn_set_option(B.OPT_XNOR_PATH, B.PATH_AUTO) == 1
    assert rc("bnn_set_option", 9, 0) == -1 and rc("bnn_set_option", 2, 4) == -1
    assert B.bnn_set_option(B.OPT_SMALL_BATCH, 0) == 1 and B.bnn_set_option(B.OPT_SMALL_BATCH, 1) == 0
    assert rc("bnn_set_option", 4, 2) == -1
    assert rc("bnn_fold_thresholds", None, None, 4, 4, 0, None, fake, None) == 1


def test_model_validation(lib):
    from paper_1706_09453_b200 import binding as B
    fake = 0x10000
    def layer(kind, k, n, act=0):
        l = B.Layer()
        l.kind, l.K, l.N, l.act = kind, k, n, act
        l.Wp, l.ldwp, l.W, l.ldw = fake, B.packed_pitch(k), fake, k
        l.thr, l.flip = fake, fake
        return l
    def model(*ls):
        arr = (B.Layer * len(ls))(*ls)
        return B.Model(len(ls), 0, arr), arr
    good, keep = model(layer(0, 440, 64, 1), layer(1, 64, 64, 1), layer(2, 64, 10))
    ws = lib.bnn_forward_workspace_bytes(C.byref(good), 8)
    assert ws >= 2 * 8 * 4 * 4
    # workspace too small / missing
    assert B.raw_call("bnn_forward", C.byref(good), fake, 440, 8, fake, 10, None, 0, None, None) == 5
    # XNOR directly on the real-valued input is not a legal chain
    bad, keep2 = model(layer(1, 440, 64, 1), layer(2, 64, 10))
    assert lib.bnn_forward_workspace_bytes(C.byref(bad), 8) == 0
    assert B.raw_call("bnn_forward", C.byref(bad), fake, 440, 8, fake, 10, fake, 1 << 20, None, None) == 4
    # fan-in mismatch
    bad, keep3 = model(layer(0, 440, 64, 1), layer(1, 32, 64, 1), layer(2, 64, 10))
    assert B.raw_call("bnn_forward", C.byref(bad), fake, 440, 8, fake, 10, fake, 1 << 20, None, None) == 2
    # unknown activation values
    odd, keep5 = model(layer(0, 440, 64, 1), layer(1, 64, 64, 1), layer(2, 64, 10))
    odd.act_values = 7
    assert B.raw_call("bnn_forward", C.byref(odd), fake, 440, 8, fake, 10, fake, 1 << 20, None, None) == 4
    # last layer must be the real-valued one
    bad, keep4 = model(layer(0, 440, 64, 1), layer(1, 64, 64, 1))
    assert B.raw_call("bnn_forward", C.byref(bad), fake, 440, 8, fake, 10, fake, 1 << 20, None, None) == 4
    # a misaligned layer_out entry of a LATER layer is refused before anything is launched
    # (0x10000 is not device memory: a launch of the first layer would have failed otherwise)
    lo = (C.c_void_p * 2)(None, fake + 4)
    assert B.raw_call("bnn_forward", C.byref(good), fake, 440, 8, fake, 10, fake, 1 << 20, lo, None) == 3
    # the new status and option entry points
    assert B.raw_call("bnn_query_status", None, None) == 1
    assert B.status_string(7) != B.status_string(6)
    assert B.raw_call("bnn_set_option", 6, 0) == -1      # wait limit: at least one microsecond
    assert B.raw_call("bnn_set_option", 5, 2) == -1      # stacking: 0 or 1
    assert B.raw_call("bnn_set_option", 7, 2) == -1      # log-softmax behind the top layer: 0 or 1
    assert B.bnn_set_option(B.OPT_SOFTMAX_FOLLOW, 0) == 1 and B.bnn_set_option(B.OPT_SOFTMAX_FOLLOW, 1) == 0
