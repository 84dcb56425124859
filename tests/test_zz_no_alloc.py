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
    # different batches and sizes, so the second call really overwrites the first one's scratch
    for frames, seed in ((256, 0), (131, 7)):
        X = model.to_dev(wl.make_frames(cfg, frames, seed=seed))
        want = dn.forward(X).clone()
        got = torch.full((frames, cfg.classes), float("nan"), dtype=torch.float32, device="cuda:0")
        B.bnn_forward_static(dn.desc, X, got)
        torch.cuda.synchronize()
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
