"""The allocation-free forward pass (bnn_forward_static) must give what bnn_forward gives.

Some users of this library may not allocate device memory while they run (a decoder thread
that must not stall, a plug-in with a fixed memory budget), so this entry point keeps its
scratch in a fixed array inside the library.  The test calls it through the C ABI twice in a
row -- the second call finds the first call's leftovers in the shared array -- and compares
with the ordinary entry point, whose scratch the caller allocates.  It sits in a file that is
collected last so that a run stopping at the first failure has already run everything else."""
import numpy as np
import pytest

from paper_1706_09453_b200 import workloads as wl

pytestmark = pytest.mark.gpu

LOGP_TOL = 1e-4   # the tolerance of the other log-probability tests


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available()
    from paper_1706_09453_b200 import build, binding, model
    build.build()
    return torch, binding, model


def test_static_forward_matches_forward_on_two_calls_in_a_row(env):
    torch, B, model = env
    cfg = wl.CONFIGS["tiny"]
    dn = model.DeviceNet(wl.make_model(cfg))
    # The first call on a device does the set-up (it looks up the array's address, and the CUDA
    # runtime may load the library's device code -- the array with it -- only then): made here, once.
    X0 = model.to_dev(wl.make_frames(cfg, 8, seed=1))
    B.bnn_forward_static(dn.desc, X0, torch.empty((8, cfg.classes), dtype=torch.float32, device="cuda:0"))
    # different batches and sizes, so the second call really overwrites the first one's scratch
    for frames, seed in ((256, 0), (131, 7)):
        X = model.to_dev(wl.make_frames(cfg, frames, seed=seed))
        want = dn.forward(X).clone()
        got = torch.full((frames, cfg.classes), float("nan"), dtype=torch.float32, device="cuda:0")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.bnn_forward_static(dn.desc, X, got)
        torch.cuda.synchronize()
        # the property the entry point exists for: the device's free memory did not move
        assert torch.cuda.mem_get_info()[0] == free_before
        err = (got - want).abs().max().item()
        assert err <= LOGP_TOL, err
        assert B.bnn_device_status() == 0


def test_static_forward_rejects_batches_beyond_its_array(env):
    torch, B, model = env
    cfg = wl.CONFIGS["tiny"]
    dn = model.DeviceNet(wl.make_model(cfg))
    frames = 40000   # 40000 x 128 B x 2 buffers > 8 MiB
    assert dn.desc.min_workspace_bytes(frames) > B.STATIC_WORKSPACE_BYTES
    X = torch.zeros((frames, cfg.in_dim), dtype=torch.float32, device="cuda:0")
    out = torch.zeros((frames, cfg.classes), dtype=torch.float32, device="cuda:0")
    with pytest.raises(B.BnnError) as e:
        B.bnn_forward_static(dn.desc, X, out)
    assert e.value.status == 5
    assert not out.any()   # nothing was launched


def test_static_forward_accepts_exactly_what_fits(env):
    """The largest batch whose scratch fits the array is accepted and correct; one frame more is
    refused with BNN_ERR_WORKSPACE.  Once for the network with binary activations and once for the
    one that hands fp32 activations from layer to layer (whose scratch per frame is 32 times larger)."""
    torch, B, model = env
    for name in ("tiny", "wsj_bw"):
        cfg = wl.CONFIGS[name]
        dn = model.DeviceNet(wl.make_model(cfg))
        lo, hi = 1, 1 << 20          # largest M with min_workspace_bytes(M) <= the array
        while lo < hi:
            mid = (lo + hi + 1) // 2
            if dn.desc.min_workspace_bytes(mid) <= B.STATIC_WORKSPACE_BYTES:
                lo = mid
            else:
                hi = mid - 1
        frames = lo
        assert dn.desc.min_workspace_bytes(frames + 1) > B.STATIC_WORKSPACE_BYTES
        X = model.to_dev(wl.make_frames(cfg, frames, seed=3))
        want = dn.forward(X).clone()
        got = torch.full((frames, cfg.classes), float("nan"), dtype=torch.float32, device="cuda:0")
        B.bnn_forward_static(dn.desc, X, got)
        torch.cuda.synchronize()
        assert (got - want).abs().max().item() <= LOGP_TOL, name
        X1 = torch.zeros((frames + 1, cfg.in_dim), dtype=torch.float32, device="cuda:0")
        out1 = torch.zeros((frames + 1, cfg.classes), dtype=torch.float32, device="cuda:0")
        with pytest.raises(B.BnnError) as e:
            B.bnn_forward_static(dn.desc, X1, out1)
        assert e.value.status == 5 and not out1.any()
        del X, X1, want, got, out1
    assert B.bnn_device_status() == 0
