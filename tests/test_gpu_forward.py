"""End-to-end parity of bnn_forward (one C-ABI call) with the CPU oracle on the synthetic
WSJ / AMI shaped networks.

The first layer is floating point: a unit whose pre-activation lies inside the float
tolerance band (|y_hat| <= 1e-4 * |scale| * sum|x_i|) may legitimately binarise either way.
So: (1) outside the band the first-layer bits must equal the oracle's; (2) the oracle then
continues from the bits the GPU actually produced, and from there on every packed bit of
every hidden layer must be identical and the log-probabilities within 1e-4."""
import numpy as np
import pytest

from oracle import bnn_oracle as o
from paper_1706_09453_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FLOAT_TOL = 1e-4
LOGP_TOL = 1e-4


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available()
    from paper_1706_09453_b200 import build, binding, model
    build.build()
    return torch, binding, model


def run_binary_net(env, cfg, frames, mode=0, sample=None, prepare_xnor=True, values=0, minimal_workspace=False):
    """Runs bnn_forward on `frames` frames; compares the frames in `sample` (all if None)."""
    torch, B, model = env
    net = wl.make_model(cfg)
    X = wl.make_frames(cfg, frames)
    dn = model.DeviceNet(net, mode, prepare_xnor=prepare_xnor, act_values=values)
    outs = dn.layer_out_buffers(frames)
    if minimal_workspace:
        small = torch.empty(dn.desc.min_workspace_bytes(frames), dtype=torch.uint8, device="cuda:0")
        assert small.numel() < dn.desc.workspace_bytes(frames)
        logp = torch.empty((frames, cfg.classes), dtype=torch.float32, device="cuda:0")
        B.bnn_forward(dn.desc, model.to_dev(X), logp, small, layer_out=outs)
    else:
        logp = dn.forward(model.to_dev(X), layer_out=outs)
    torch.cuda.synchronize()
    idx = np.arange(frames) if sample is None else np.asarray(sample)
    gbits = [model.words_to_numpy(t, cfg.hidden)[idx] for t in outs]
    glogp = logp.cpu().numpy()[idx]
    # the packed weights themselves (Eq. 3 on the GPU) must equal the oracle's
    ref = o.forward(X[idx], net.W, net.scale, net.shift, net.Wout, net.bout, o.ACT_SIGN, mode,
                    layer1_bits=gbits[0], values=values)
    for l, wp in enumerate(dn.Wp):
        np.testing.assert_array_equal(model.words_to_numpy(wp, net.W[l].shape[1]), ref["Wp"][l])
    # (1) first layer: equal outside the tolerance band
    yh = ref["pre"][0]
    band = FLOAT_TOL * np.abs(net.scale[0])[None, :] * ref["sumabs"][:, None]
    own = o.unpack_pm1(ref["bits_own_layer1"], cfg.hidden)
    got = o.unpack_pm1(gbits[0], cfg.hidden)
    decided = np.abs(yh) > band
    np.testing.assert_array_equal(got[decided], own[decided])
    ambiguous = 1.0 - decided.mean()
    assert ambiguous < 5e-3, ambiguous
    # (2) everything downstream of the GPU's own first-layer bits is bit-exact
    for l in range(1, cfg.n_hidden):
        np.testing.assert_array_equal(gbits[l], ref["bits"][l], err_msg="hidden layer %d" % (l + 1))
    err = np.abs(glogp - ref["logp"]).max()
    assert err <= LOGP_TOL, err
    return dict(ambiguous=ambiguous, flipped=float((got != own).mean()), logp_err=float(err))


def test_forward_tiny_config_all_frames(env):
    r = run_binary_net(env, wl.CONFIGS["tiny"], 256)
    assert r["flipped"] <= r["ambiguous"]
    assert env[1].bnn_device_status() == 0


def test_forward_tiny_config_weights_widened_on_the_fly(env):
    """The model without prepared images of the hidden layers' weights (bnn_xnor_gemm's kernel)."""
    run_binary_net(env, wl.CONFIGS["tiny"], 256, prepare_xnor=False)


def test_forward_tiny_config_01_activations(env):
    """Hidden activations in (0,1) instead of (-1,+1) (Section 3.2), on every XNOR kernel."""
    B = env[1]
    run_binary_net(env, wl.CONFIGS["tiny"], 256, values=1)
    run_binary_net(env, wl.CONFIGS["tiny"], 200, values=1, prepare_xnor=False, mode=1)
    prev = B.bnn_set_xnor_path(B.XNOR_POPC)
    try:
        run_binary_net(env, wl.CONFIGS["tiny"], 131, values=1)
    finally:
        B.bnn_set_xnor_path(prev)
    assert B.bnn_device_status() == 0


def test_forward_wsj_config_01_activations_sampled_frames(env):
    cfg = wl.CONFIGS["wsj"]
    rng = np.random.default_rng(2)
    sample = np.unique(np.concatenate([np.arange(64), np.arange(cfg.frames - 64, cfg.frames),
                                       rng.integers(0, cfg.frames, 200)]))
    run_binary_net(env, cfg, cfg.frames, sample=sample, values=1)


def test_forward_tiny_config_popcount_path(env):
    B = env[1]
    prev = B.bnn_set_xnor_path(B.XNOR_POPC)
    try:
        run_binary_net(env, wl.CONFIGS["tiny"], 256)
    finally:
        B.bnn_set_xnor_path(prev)


def test_forward_tiny_config_paper_sign_convention(env):
    run_binary_net(env, wl.CONFIGS["tiny"], 256, mode=1)


def test_forward_ragged_frame_count(env):
    run_binary_net(env, wl.CONFIGS["tiny"], 131)


def test_forward_single_frame(env):
    run_binary_net(env, wl.CONFIGS["tiny"], 1)


def test_forward_small_batch_at_the_edge_of_the_staging_memory(env):
    """16 frames and a fan-in of 768: the staged operand of the matrix-vector kernels (16 x 768 floats =
    48 KB) no longer fits next to their static arrays, so the forward pass must take the tiled kernels
    instead of failing at launch; 752 still fits the matrix-vector kernels."""
    import dataclasses
    for in_dim in (752, 768):
        cfg = dataclasses.replace(wl.CONFIGS["tiny"], in_dim=in_dim)
        run_binary_net(env, cfg, 16)
    assert env[1].bnn_device_status() == 0


@pytest.mark.parametrize("hidden,n_hidden,frames,values", [
    (1000, 4, 700, 0),     # units and fan-in not multiples of the tile / stage sizes (ragged last stage)
    (1280, 3, 1500, 1),    # odd number of K stages; (0,1) activations
    (96, 5, 300, 0),       # a single, narrow unit tile
    (512, 11, 400, 0),     # ten binary layers in a row: more than one launch can hold, so two runs
])
def test_forward_stacked_hidden_layers_edge_shapes(env, hidden, n_hidden, frames, values):
    """The run of binary hidden layers as one launch on shapes that exercise its tails, checked against
    the oracle like every other network (and once more with one launch per layer)."""
    import dataclasses
    B = env[1]
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], hidden=hidden, n_hidden=n_hidden, classes=300)
    run_binary_net(env, cfg, frames, values=values)
    prev = B.bnn_set_option(B.OPT_XNOR_STACK, 0)
    try:
        run_binary_net(env, cfg, frames, values=values)
    finally:
        B.bnn_set_option(B.OPT_XNOR_STACK, prev)
    assert B.bnn_device_status() == 0


@pytest.mark.parametrize("frames,classes,values,with_prior", [
    (2100, 4000, 0, False),   # 5 frame groups x 32 class tiles, ragged last group, the wide-row variant
    (4700, 2000, 1, True),    # 10 groups x 16 class tiles, the narrow-row variant; (0,1) activations; log-prior
    (2561, 3400, 0, True),    # one frame in the last group
    (2100, 4100, 0, False),   # more classes than the following kernel holds in registers: the kernels run one after the other
])
def test_forward_log_softmax_following_the_top_layer(env, frames, classes, values, with_prior):
    """The log-softmax launched behind the top layer's kernel, taking each group of 512 frames as soon as
    its logits are complete (default when the top layer has more than one wave of tiles), against the
    oracle, against the two kernels run one after the other, and repeated into the same workspace."""
    import dataclasses
    torch, B, model = env
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], hidden=256, n_hidden=2, classes=classes)
    net = wl.make_model(cfg)
    X = wl.make_frames(cfg, frames)
    rng = np.random.default_rng(frames)
    log_prior = np.log(rng.dirichlet(np.ones(classes) * 5.0)).astype(np.float32) if with_prior else None
    dn = model.DeviceNet(net, act_values=values, log_prior=log_prior)
    outs = dn.layer_out_buffers(frames)
    Xd = model.to_dev(X)
    a = dn.forward(Xd, layer_out=outs).clone()
    g1 = model.words_to_numpy(outs[0], cfg.hidden)
    ref = o.forward(X, net.W, net.scale, net.shift, net.Wout, net.bout, o.ACT_SIGN, 0, layer1_bits=g1,
                    values=values, log_prior=log_prior)
    assert np.abs(a.cpu().numpy() - ref["logp"]).max() <= LOGP_TOL
    prev = B.bnn_set_option(B.OPT_SOFTMAX_FOLLOW, 0)
    try:
        b = dn.forward(Xd, layer_out=outs).clone()
    finally:
        B.bnn_set_option(B.OPT_SOFTMAX_FOLLOW, prev)
    assert prev == 1
    # the same arithmetic per element; only the order of the row reductions differs
    assert (a - b).abs().max().item() <= 1e-5
    for _ in range(3):   # the counters are cleared by every call
        assert torch.equal(dn.forward(Xd), a)
    # rows of the output that are not 16-byte aligned: the following kernel does not apply, same result
    wide = torch.full((frames, classes + 3), 7.0, dtype=torch.float32, device="cuda:0")
    c = dn.forward(Xd, logp=wide[:, :classes])
    assert (c - a).abs().max().item() <= 1e-5
    assert bool((wide[:, classes:] == 7.0).all())
    assert B.bnn_device_status() == 0


def test_forward_wsj_config_full_batch_sampled_frames(env):
    """The benchmark's launch configuration (8192 frames); the oracle checks 600 of them,
    including the first and last tile of frames."""
    cfg = wl.CONFIGS["wsj"]
    rng = np.random.default_rng(0)
    sample = np.unique(np.concatenate([np.arange(128), np.arange(cfg.frames - 128, cfg.frames),
                                       rng.integers(0, cfg.frames, 344)]))
    run_binary_net(env, cfg, cfg.frames, sample=sample)


def test_forward_ami_config_full_batch_sampled_frames(env):
    cfg = wl.CONFIGS["ami"]
    rng = np.random.default_rng(1)
    sample = np.unique(np.concatenate([np.arange(128), np.arange(cfg.frames - 128, cfg.frames),
                                       rng.integers(0, cfg.frames, 1024)]))
    run_binary_net(env, cfg, cfg.frames, sample=sample)


def test_forward_minimal_workspace_against_the_oracle(env):
    """With only the minimal scratch the first layer runs without the split-activation image (its
    kernel splits inside the GEMM): the same procedure against the oracle as with the full scratch."""
    run_binary_net(env, wl.CONFIGS["tiny"], 200, minimal_workspace=True)
    assert env[1].bnn_device_status() == 0


def test_forward_one_launch_per_hidden_layer_gives_the_same_bits(env):
    """The run of equal binary hidden layers as one launch (default) and as one launch per layer:
    identical bits in every layer and identical log-probabilities, at a size where every CTA of the
    stacked launch has several frame tiles and the layers overlap."""
    torch, B, model = env
    cfg = wl.CONFIGS["wsj"]
    frames = 4000 + 37
    dn = model.DeviceNet(wl.make_model(cfg))
    X = model.to_dev(wl.make_frames(cfg, frames))
    outs_a, outs_b = dn.layer_out_buffers(frames), dn.layer_out_buffers(frames)
    a = dn.forward(X, layer_out=outs_a).clone()
    prev = B.bnn_set_option(B.OPT_XNOR_STACK, 0)
    try:
        b = dn.forward(X, layer_out=outs_b).clone()
    finally:
        B.bnn_set_option(B.OPT_XNOR_STACK, prev)
    for l, (ta, tb) in enumerate(zip(outs_a, outs_b)):
        nw = (cfg.hidden + 31) // 32
        assert torch.equal(ta[:, :nw], tb[:, :nw]), "layer %d" % (l + 1)
    assert torch.equal(a, b)
    # repeated launches into the workspace (no layer_out): the counters are cleared by every call
    ref = dn.forward(X).clone()
    for _ in range(5):
        assert torch.equal(dn.forward(X), ref)
    assert torch.equal(ref, a)
    assert B.bnn_device_status() == 0


def test_forward_unwritten_workspace_path_equals_layer_out_path(env):
    """Without layer_out the activations go through the workspace: same log-probabilities."""
    torch, B, model = env
    cfg = wl.CONFIGS["tiny"]
    dn = model.DeviceNet(wl.make_model(cfg))
    X = model.to_dev(wl.make_frames(cfg, 200))
    a = dn.forward(X).clone()
    b = dn.forward(X, layer_out=dn.layer_out_buffers(200))
    assert torch.equal(a, b)


def test_forward_binary_weights_only_chained_images_equal_fp32_hand_over(env):
    """Binary weights, real activations: without layer_out every hidden layer writes the next layer's
    split-activation image directly; with layer_out it also stores fp32 rows.  Both, and the minimal
    scratch (fp32 rows, split again by every layer), give the same log-probabilities bit for bit: the
    bf16 terms are the same numbers however they get into the image."""
    torch, B, model = env
    cfg = wl.CONFIGS["wsj_bw"]
    frames = 300
    dn = model.DeviceNet(wl.make_model(cfg))
    X = model.to_dev(wl.make_frames(cfg, frames))
    a = dn.forward(X).clone()
    b = dn.forward(X, layer_out=dn.layer_out_buffers(frames)).clone()
    assert torch.equal(a, b)
    small = torch.empty(dn.desc.min_workspace_bytes(frames), dtype=torch.uint8, device="cuda:0")
    c = torch.empty_like(a)
    B.bnn_forward(dn.desc, X, c, small)
    assert (a - c).abs().max().item() <= LOGP_TOL
    assert B.bnn_device_status() == 0


def test_forward_mixed_topology_sigmoid_units_into_the_top_layers_image(env):
    """The binary layer with Sigmoid units feeds the real-valued top layer: without layer_out its
    Sigmoid outputs go straight into the top layer's image of fp16 terms, with layer_out through fp32
    rows that are split afterwards.  The terms are the same numbers, so the log-probabilities are equal."""
    torch, B, model = env
    cfg = wl.CONFIGS["wsj_mixed"]
    frames = 300
    dn = model.DeviceNet(wl.make_model(cfg))
    X = model.to_dev(wl.make_frames(cfg, frames))
    a = dn.forward(X).clone()
    b = dn.forward(X, layer_out=dn.layer_out_buffers(frames)).clone()
    assert torch.equal(a, b)
    assert B.bnn_device_status() == 0


def run_bw_net(env, cfg, frames, sample=None):
    torch, B, model = env
    net = wl.make_model(cfg)
    X = wl.make_frames(cfg, frames)
    dn = model.DeviceNet(net)
    outs = dn.layer_out_buffers(frames)
    logp = dn.forward(model.to_dev(X), layer_out=outs)
    torch.cuda.synchronize()
    idx = np.arange(frames) if sample is None else np.asarray(sample)
    ref = o.forward(X[idx], net.W, net.scale, net.shift, net.Wout, net.bout, o.ACT_HARDTANH)
    # per-layer, teacher-forced: layer l of the GPU is fed the oracle's layer l-1 output
    prev = X[idx]
    for l in range(cfg.n_hidden):
        y = torch.empty((len(idx), cfg.hidden), dtype=torch.float32, device="cuda:0")
        B.bnn_signw_gemm(model.to_dev(prev), dn.Wp[l], net.W[l].shape[1], Y=y, act=B.ACT_HARDTANH,
                         scale=dn.scale[l], shift=dn.shift[l])
        tol = FLOAT_TOL * np.abs(net.scale[l])[None, :] * ref["sumabs_l"][l][:, None]
        assert (np.abs(y.cpu().numpy() - ref["h"][l]) <= tol).all(), l
        prev = ref["h"][l].astype(np.float32)
    # end to end
    err = np.abs(logp.cpu().numpy()[idx] - ref["logp"]).max()
    assert err <= LOGP_TOL, err
    herr = np.abs(outs[-1].cpu().numpy()[idx] - ref["h"][-1]).max()
    assert herr <= 1e-4, herr


def test_forward_binary_weights_only_small(env):
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["wsj_bw"], hidden=512, classes=700, frames=200)
    run_bw_net(env, cfg, 200)


def test_forward_binary_weights_only_wsj_config_sampled(env):
    cfg = wl.CONFIGS["wsj_bw"]
    rng = np.random.default_rng(2)
    sample = np.unique(np.concatenate([np.arange(64), np.arange(cfg.frames - 64, cfg.frames),
                                       rng.integers(0, cfg.frames, 128)]))
    run_bw_net(env, cfg, cfg.frames, sample=sample)


@pytest.mark.parametrize("frames", [300, 3])
def test_forward_spliced_input_and_log_prior(env, frames):
    """The context window formed inside the first layer (one 40-dim frame per input row, 5 + 1 + 5
    frames of context, edge frames repeated) and the log-prior subtracted after the log-softmax:
    equal to the oracle run on the explicitly spliced input."""
    torch, B, model = env
    cfg = wl.CONFIGS["tiny"]
    net = wl.make_model(cfg)
    rng = np.random.default_rng(frames)
    F = rng.standard_normal((frames, 40)).astype(np.float32)
    prior = rng.dirichlet(np.ones(cfg.classes) * 5.0)
    log_prior = np.log(prior).astype(np.float32)
    dn = model.DeviceNet(net, splice=(5, 5), log_prior=log_prior)
    outs = dn.layer_out_buffers(frames)
    Fd = torch.full((frames, 44), 7.0, dtype=torch.float32, device="cuda:0")   # pitch 44: 16-byte aligned rows
    Fd[:, :40] = model.to_dev(F)
    logp = dn.forward(Fd[:, :40], layer_out=outs)
    torch.cuda.synchronize()
    X = o.splice(F, 5, 5)
    assert X.shape == (frames, cfg.in_dim)
    g1 = model.words_to_numpy(outs[0], cfg.hidden)
    ref = o.forward(X, net.W, net.scale, net.shift, net.Wout, net.bout, o.ACT_SIGN, 0, layer1_bits=g1,
                    log_prior=log_prior)
    band = FLOAT_TOL * np.abs(net.scale[0])[None, :] * ref["sumabs"][:, None]
    decided = np.abs(ref["pre"][0]) > band
    np.testing.assert_array_equal(o.unpack_pm1(g1, cfg.hidden)[decided],
                                  o.unpack_pm1(ref["bits_own_layer1"], cfg.hidden)[decided])
    assert decided.mean() > 0.995
    for l in range(1, cfg.n_hidden):
        np.testing.assert_array_equal(model.words_to_numpy(outs[l], cfg.hidden), ref["bits"][l])
    assert np.abs(logp.cpu().numpy() - ref["logp"]).max() <= LOGP_TOL
    # an unaligned pitch takes the scalar path of the splitting kernel: same bits
    Fu = torch.full((frames, 41), 7.0, dtype=torch.float32, device="cuda:0")
    Fu[:, :40] = model.to_dev(F)
    outs2 = dn.layer_out_buffers(frames)
    logp2 = dn.forward(Fu[:, :40], layer_out=outs2)
    assert torch.equal(outs2[0], outs[0]) and torch.equal(logp2, logp)
    # the window needs the scratch image: the minimal workspace is refused
    small = torch.empty(dn.desc.min_workspace_bytes(frames), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.BnnError) as e:
        B.bnn_forward(dn.desc, Fd[:, :40], logp, small)
    assert e.value.status == 5
    assert B.bnn_device_status() == 0


def run_mixed_net(env, cfg, frames, sample=None, mode=0):
    """The paper's mixed topology through bnn_forward: real-valued Sigmoid first layer, +-1 weights
    with Sign units, +-1 x +-1 with Sign units, +-1 x +-1 with Sigmoid units, real Softmax layer."""
    torch, B, model = env
    net = wl.make_model(cfg)
    X = wl.make_frames(cfg, frames)
    dn = model.DeviceNet(net, mode)
    outs = dn.layer_out_buffers(frames)
    logp = dn.forward(model.to_dev(X), layer_out=outs)
    torch.cuda.synchronize()
    idx = np.arange(frames) if sample is None else np.asarray(sample)
    g2 = model.words_to_numpy(outs[1], cfg.hidden)[idx]
    ref = o.forward_mixed(X[idx], net.W, net.scale, net.shift, net.Wout, net.bout, mode, layer2_bits=g2)
    # layer 1: Sigmoid units; the pre-activation is within 2^-17 sum|x||w| and |d sigmoid| <= |dz| / 4
    bound = 0.25 * 2.0 ** -17 * (np.abs(X[idx]).astype(np.float64) @ np.abs(net.W[0]).astype(np.float64).T) + 2e-7
    assert (np.abs(outs[0].cpu().numpy()[idx] - ref["h1"]) <= bound).all()
    # layer 2: bits equal outside the float tolerance band
    band = FLOAT_TOL * np.abs(net.scale[1])[None, :] * ref["sumabs2"][:, None]
    decided = np.abs(ref["pre2"]) > band
    np.testing.assert_array_equal(o.unpack_pm1(g2, cfg.hidden)[decided],
                                  o.unpack_pm1(ref["bits_own_layer2"], cfg.hidden)[decided])
    assert decided.mean() > 0.99, decided.mean()
    # downstream of the GPU's own layer-2 bits: binary layers bit-exact, Sigmoid units and log-probs close
    for l in range(2, cfg.n_hidden - 1):
        np.testing.assert_array_equal(model.words_to_numpy(outs[l], cfg.hidden)[idx], ref["bits"][l - 1])
    assert np.abs(outs[-1].cpu().numpy()[idx] - ref["hL"]).max() <= 1e-6
    err = np.abs(logp.cpu().numpy()[idx] - ref["logp"]).max()
    assert err <= LOGP_TOL, err
    assert B.bnn_device_status() == 0


def test_forward_mixed_topology_small(env):
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["wsj_mixed"], hidden=512, classes=700, frames=300, n_hidden=4)
    run_mixed_net(env, cfg, 300)
    run_mixed_net(env, cfg, 77, mode=1)


def test_forward_mixed_topology_wsj_shape_sampled(env):
    cfg = wl.CONFIGS["wsj_mixed"]
    rng = np.random.default_rng(3)
    sample = np.unique(np.concatenate([np.arange(64), np.arange(cfg.frames - 64, cfg.frames),
                                       rng.integers(0, cfg.frames, 128)]))
    run_mixed_net(env, cfg, cfg.frames, sample=sample)


@pytest.mark.parametrize("frames", [1, 5, 16])
@pytest.mark.parametrize("values", [0, 1])
def test_forward_small_batch_kernels(env, frames, values):
    """Batches of up to 16 frames run on the matrix-vector kernels (one warp per unit): same parity
    with the oracle as the tiled kernels, for both activation value sets and both Sign conventions,
    and on sizes that are not multiples of 32."""
    import dataclasses
    B = env[1]
    assert B.bnn_set_option(B.OPT_SMALL_BATCH, 1) in (0, 1)
    run_binary_net(env, wl.CONFIGS["tiny"], frames, values=values)
    odd = dataclasses.replace(wl.CONFIGS["tiny"], hidden=1000, classes=3307, in_dim=441)
    run_binary_net(env, odd, frames, values=values, mode=1)
    # the tiled kernels on the same batch (option off) still agree with the oracle
    prev = B.bnn_set_option(B.OPT_SMALL_BATCH, 0)
    try:
        run_binary_net(env, wl.CONFIGS["tiny"], frames, values=values)
    finally:
        B.bnn_set_option(B.OPT_SMALL_BATCH, prev)
    assert B.bnn_device_status() == 0


def test_forward_small_batch_other_topologies(env):
    """A few frames through the networks whose layers only partly have matrix-vector kernels
    (fp32 activations, Sigmoid units): small and tiled kernels chain on the same buffers."""
    import dataclasses
    bw = dataclasses.replace(wl.CONFIGS["wsj_bw"], hidden=512, classes=700, frames=5)
    run_bw_net(env, bw, 5)
    mixed = dataclasses.replace(wl.CONFIGS["wsj_mixed"], hidden=512, classes=700, frames=7, n_hidden=4)
    run_mixed_net(env, mixed, 7)
    run_mixed_net(env, wl.CONFIGS["wsj_mixed"], 3)
