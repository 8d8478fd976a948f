"""GPU parity of the whole DDG iteration: CUDA library vs CPU oracle, step by step, through the C ABI.
Tolerances: fp32 mode 1e-4 relative per tensor (gradients, weights) and 1e-3 on the loss trajectory; bf16 mode
2e-2 relative against the oracle with the same bf16 storage points."""
import numpy as np
import pytest
import torch

from paper_1804_10574_b200 import nets
from tests.parity import rel, run_pair  # noqa: F401

pytestmark = pytest.mark.gpu

FP32_TOL, BF16_TOL, LOSS_TOL = 1e-4, 2e-2, 1e-3
RATIO_BAND = (0.85, 1.2)       # median of rel(gpu, exact) / rel(oracle_bf16, exact) over gradient tensors


def test_mlp_k2_20_steps_fp32():
    """Config 1.  Also against the exact oracle (no storage rounding anywhere): a network this small meets no ReLU
    pre-activation within fp32 rounding of zero, so the fp32 path stays within the fp32 bar of the exact run too."""
    w = run_pair(nets.config("mlp"), 20, FP32_TOL, LOSS_TOL, exact_too=True)
    print("mlp K=2 worst", w)
    assert w["grad_vs_exact"] <= FP32_TOL and w["weight_vs_exact"] <= FP32_TOL


@pytest.mark.parametrize("splits", [[], [0], [0, 1, 2]], ids=["K1", "K2_early", "K4"])
def test_mlp_other_splits_fp32(splits):
    run_pair(nets.config("mlp"), 8, FP32_TOL, LOSS_TOL, split_after=splits)


def test_mlp_ragged_batch_and_momentum_fp32():
    cfg = dict(nets.config("mlp"), opt=dict(lr=0.05, momentum=0.9, weight_decay=1e-3))
    run_pair(cfg, 8, FP32_TOL, LOSS_TOL, batch=7)


def test_mlp_k2_bf16():
    """Config 1 in the bf16 mode: every layer runs on the tensor-core FC kernels (forward, and dx / dW / db in one
    launch).  A four-layer network stores few tensors, so the plain bf16 tolerance applies."""
    w = run_pair(nets.config("mlp"), 10, BF16_TOL, 5e-3, precision="bf16")
    print("mlp bf16 worst", w)


def test_mlp_adam_fp32():
    cfg = dict(nets.config("mlp"), opt=dict(lr=1e-3, momentum=0.0, weight_decay=0.0))
    run_pair(cfg, 8, FP32_TOL, LOSS_TOL, opt="adam")


def test_mlp_diminishing_stepsize_fp32():
    run_pair(nets.config("mlp"), 6, FP32_TOL, LOSS_TOL, lr_schedule=lambda t: 0.05 / (1 + t))


def test_resnet8_k2_20_steps_fp32():
    """Config 2.  Bit-level agreement is with the oracle that stores fp32 where the kernels do.  The exact oracle (no
    storage rounding) is run beside it for the record: of the 2.4 M ReLU decisions per iteration the few whose
    pre-activation lies within fp32 rounding of zero fall differently in an fp32-storage and an fp64 run, each such
    event moves these cancellation-dominated gradients by a per cent or so, and lr 0.1 with momentum 0.9 amplifies it:
    after 20 iterations single gradient tensors of the two ORACLE runs differ by tens of per cent while the loss
    trajectories stay within 1e-3 (seen: 9.4e-4) - no fp32 path can be within 1e-4 of the exact run here, which is why
    the per-step bar is taken against the fp32-storage oracle.  test_resnet8_first_steps_fp32_vs_exact holds the exact
    oracle to the fp32 bar where that is possible."""
    w = run_pair(nets.config("resnet8"), 20, FP32_TOL, LOSS_TOL, exact_too=True, exact_loss_tol=3e-3)
    print("resnet8 K=2 worst", w)
    assert w["weight_vs_exact"] <= 0.1


def test_resnet8_first_steps_fp32_vs_exact():
    """Where no ReLU pre-activation falls within fp32 rounding of zero (batch 4: 0.3 M decisions per iteration instead of
    2.4 M; three iterations from identical weights) the fp32 path is within the fp32 bar of the exact oracle as well.  At
    batch 32 the first such event already falls inside the first three iterations (seen: one gradient tensor 1.4e-2 off
    while the weights are still within 6e-5)."""
    w = run_pair(nets.config("resnet8"), 3, FP32_TOL, LOSS_TOL, exact_too=True, batch=4)
    print("resnet8 first steps vs exact", w)
    assert w["grad_vs_exact"] <= FP32_TOL and w["weight_vs_exact"] <= FP32_TOL


@pytest.mark.parametrize("net,splits,batch", [("mlp", [0, 1], 16), ("mlp", [0, 1, 2], 16), ("resnet8", [1, 2, 3], 4)],
                         ids=["mlp_K3", "mlp_K4", "resnet8_K4"])
def test_graph_replay_over_two_ring_periods_fp32(net, splits, batch):
    """Every recorded piece is replayed at least twice more after its recording: K-1 warm-up iterations, then two full
    ring periods (lcm(1..K, 2): 6 at K=3, 12 at K=4) and one more.  fp32 mode, so any pointer that is wrong at
    t + period shows as a bit-level difference; debug_checks adds the device-side ring stamps (the delay pattern of
    Eq. 6-8 checked on the GPU itself)."""
    K = len(splits) + 1
    period = {3: 6, 4: 12}[K]
    cfg = dict(nets.config(net), opt=dict(lr=0.02, momentum=0.9, weight_decay=5e-4))
    run_pair(cfg, K - 1 + 2 * period + 1, FP32_TOL, LOSS_TOL, split_after=splits, batch=batch, use_graph=True,
             gpu_kwargs=dict(debug_checks=True))


def test_step_size_schedule_and_adam_keep_the_graphs_fp32():
    """The step size sequence gamma_t (Theorem 2's diminishing sequence) and Adam's iteration-dependent bias corrections
    live in device memory: a run that changes the step size every iteration replays the same recordings."""
    cfg = dict(nets.config("mlp"), opt=dict(lr=0.05, momentum=0.9, weight_decay=0.0))
    run_pair(cfg, 12, FP32_TOL, LOSS_TOL, use_graph=True, lr_schedule=lambda t: 0.05 / (1 + t))
    cfg = dict(nets.config("resnet8"), opt=dict(lr=1e-3, momentum=0.0, weight_decay=0.0))
    run_pair(cfg, 8, FP32_TOL, LOSS_TOL, batch=6, opt="adam", use_graph=True, lr_schedule=lambda t: 1e-3 / (1 + 0.1 * t))


@pytest.mark.parametrize("splits", [[], [2, 3], [1, 2, 3]], ids=["K1", "K3", "K4"])
def test_resnet8_other_splits_fp32(splits):
    cfg = dict(nets.config("resnet8"), opt=dict(lr=0.05, momentum=0.9, weight_decay=5e-4))
    run_pair(cfg, 6, FP32_TOL, LOSS_TOL, split_after=splits, batch=5)


@pytest.mark.parametrize("split", [1, 2, 3, 4], ids=["after1", "after3", "after5", "after7"])
def test_resnet8_split_positions_adam_fp32(split):
    """The split-position sweep of Section 5.1: ResNet-8 cut after weighted layer 1, 3, 5, 7 (after the stem and after
    each block), trained with Adam (Algorithm 2) as there."""
    cfg = dict(nets.config("resnet8"), opt=dict(lr=1e-3, momentum=0.0, weight_decay=0.0))
    run_pair(cfg, 6, FP32_TOL, LOSS_TOL, split_after=[split], batch=6, opt="adam")


@pytest.mark.parametrize("split", [[1], [4], [1, 2, 3]], ids=["after1", "after7", "K4"])
def test_resnet8_split_positions_bf16(split):
    """The same cuts in the bf16 mode the sweep is timed in (tensor-core kernels, epilogue batch-norm sums)."""
    cfg = dict(nets.config("resnet8"), opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    run_pair(cfg, 5, BF16_TOL, 5e-3, precision="bf16", split_after=split, noise_bar=True, ratio_band=RATIO_BAND)


@pytest.mark.parametrize("splits", [[2], [2, 3]], ids=["K2", "K3"])
def test_resnet8_projection_shortcuts_fp32(splits):
    """Section 5.1's network with 1x1-projection shortcuts on the two shape-changing blocks (the second shortcut type),
    fp32 mode: bit-level parity with the oracle over two ring periods, graph replay on."""
    cfg = dict(nets.config("resnet8"), layers=nets.resnet(1, 10, projection=True), opt=dict(lr=0.05, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 14, FP32_TOL, LOSS_TOL, split_after=splits, batch=8, use_graph=True)
    print("resnet8 projection fp32 worst", w)


def test_resnet8_projection_shortcuts_bf16():
    cfg = dict(nets.config("resnet8"), layers=nets.resnet(1, 10, projection=True), opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 6, BF16_TOL, 5e-3, precision="bf16", split_after=[2, 3], noise_bar=True, ratio_band=RATIO_BAND)
    print("resnet8 projection bf16 worst", w)


@pytest.mark.parametrize("c,h,stride", [(16, 32, 2), (32, 16, 2), (16, 16, 1)], ids=["c16_s2", "c32_s2", "c16_to_32_s1"])
def test_one_projection_block_bf16(c, h, stride):
    co = 2 * c
    L = [(nets.BASIC_BLOCK_PROJ, c, co, stride, 0, 0), (nets.GLOBAL_AVGPOOL, co, co, 1, 0, 0), (nets.FC, co, 10, 1, 1, 0)]
    cfg = dict(layers=L, split_after=[], batch=32, in_shape=(c, h, h), num_classes=10, precision="bf16",
               opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 2, BF16_TOL, 5e-3)
    print("one projection block c=%d stride=%d worst" % (c, stride), w)


def test_resnet8_graph_replay_matches_fp32():
    run_pair(nets.config("resnet8"), 8, FP32_TOL, LOSS_TOL, batch=8, use_graph=True)


def test_generic_layers_fp32():
    """Stand-alone conv(+relu), bn, relu, pool layers outside basic blocks, odd sizes."""
    L = [(nets.CONV3X3, 3, 8, 1, 0, 1), (nets.BN, 8, 8, 1, 0, 0), (nets.RELU, 8, 8, 1, 0, 0),
         (nets.CONV3X3, 8, 12, 2, 0, 0), (nets.BN, 12, 12, 1, 0, 1), (nets.GLOBAL_AVGPOOL, 12, 12, 1, 0, 0),
         (nets.FC, 12, 9, 1, 1, 1), (nets.FC, 9, 5, 1, 0, 0)]
    cfg = dict(layers=L, split_after=[1, 4], batch=6, in_shape=(3, 9, 7), num_classes=5, precision="fp32",
               opt=dict(lr=0.05, momentum=0.5, weight_decay=1e-3))
    run_pair(cfg, 6, FP32_TOL, LOSS_TOL)


def test_resnet8_k2_bf16():
    cfg = dict(nets.config("resnet8"), opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 6, BF16_TOL, 5e-3, precision="bf16", noise_bar=True, ratio_band=RATIO_BAND)
    print("resnet8 bf16 worst", w)


def test_resnet20_k3_bf16_graph():
    L = nets.resnet(3, 10)
    cfg = dict(layers=L, split_after=nets.split_even_blocks(L, 3), batch=32, in_shape=(3, 32, 32), num_classes=10,
               precision="bf16", opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 8, BF16_TOL, 5e-3, use_graph=True, noise_bar=True, ratio_band=RATIO_BAND)
    print("resnet20 bf16 worst", w)


@pytest.mark.parametrize("c,h,stride", [(16, 32, 1), (32, 16, 1), (64, 8, 1), (16, 32, 2), (32, 16, 2)],
                         ids=["c16", "c32", "c64", "c16_s2", "c32_s2"])
def test_one_block_networks_bf16(c, h, stride):
    """input -> BASIC_BLOCK -> global mean pool -> FC, K = 1, per stage width and stride: the tensor-core convolutions
    with their fused epilogues (batch-norm sums, shortcut gradient) in the smallest network that contains them.  Only a
    handful of bf16 stores separate the two sides here, so the plain bf16 tolerance applies without any noise rule."""
    co = c * stride
    L = [(nets.BASIC_BLOCK, c, co, stride, 0, 0), (nets.GLOBAL_AVGPOOL, co, co, 1, 0, 0), (nets.FC, co, 10, 1, 1, 0)]
    cfg = dict(layers=L, split_after=[], batch=32, in_shape=(c, h, h), num_classes=10, precision="bf16",
               opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 2, BF16_TOL, 5e-3)
    print("one block c=%d stride=%d worst" % (c, stride), w)


def test_resnet56_k2_bf16_graph():
    """Config 3: ResNet-56 (units 9-9-9), K = 2 split at the centre (14 + 13 blocks), batch 128, bf16 storage, graph
    replay: four iterations against the oracle at full size."""
    cfg = nets.config("resnet56")
    w = run_pair(cfg, 4, BF16_TOL, 5e-3, use_graph=True, noise_bar=True, ratio_band=RATIO_BAND)
    print("resnet56 K=2 full size worst", w)


def test_create_rejects_bad_specs():
    from paper_1804_10574_b200 import binding
    L = nets.mlp()
    with pytest.raises(binding.DdgError) as e:
        binding.Ddg(L, [3], 4, (64, 1, 1), 10)            # split after the last layer
    assert e.value.status == 2
    with pytest.raises(binding.DdgError) as e:
        binding.Ddg(L, [1], 4, (63, 1, 1), 10)            # wrong input width
    assert e.value.status == 2
    with pytest.raises(binding.DdgError) as e:
        binding.Ddg(L[:-1], [1], 4, (64, 1, 1), 10)       # output is not num_classes wide
    assert e.value.status == 2
    with pytest.raises(binding.DdgError) as e:
        binding.Ddg([(nets.CONV3X3, 3, 8, 1, 1, 0), (nets.GLOBAL_AVGPOOL, 8, 8, 1, 0, 0), (nets.FC, 8, 2, 1, 1, 0)],
                    [], 2, (3, 4, 4), 2)                  # conv bias
    assert e.value.status == 3
    d = binding.Ddg(L, [1], 4, (64, 1, 1), 10)
    x = torch.zeros(4, 64, device="cuda"); y = torch.zeros(4, dtype=torch.int32, device="cuda")
    d.step(x, y)
    with pytest.raises(binding.DdgError) as e:
        d.set_weights(np.zeros(d.n_params, dtype=np.float32))   # only before the first step
    assert e.value.status == 7
    d.destroy()


def test_resnet110_k4_full_size_bf16_graph():
    """The benchmark's own configuration (ResNet-110, K=4, batch 128, bf16, graph replay, 100 classes): five
    iterations against the oracle at full size.  Every module applies its first real delayed gradient inside the
    window (delays 3, 2, 1, 0), loss and weights are held to the bf16 bars, gradients to the format-noise bar."""
    cfg = nets.config("resnet110")
    w = run_pair(cfg, 5, BF16_TOL, 5e-3, use_graph=True, noise_bar=True, ratio_band=RATIO_BAND, check_every=2)
    print("resnet110 K=4 full size worst", w)


def _resnet20_k3_bf16_run(**kw):
    from paper_1804_10574_b200 import binding, synth
    L = nets.resnet(3, 10)
    B, shape, classes = 32, (3, 32, 32), 10
    d = binding.Ddg(L, nets.split_even_blocks(L, 3), B, shape, classes, precision="bf16", lr=0.01, momentum=0.9,
                    weight_decay=5e-4, use_graph=True, **kw)
    d.set_weights(synth.init_weights(L, perturb_affine=0.1))
    losses = []
    for t in range(6):
        x, y = synth.batch(t, B, shape, classes)
        losses.append(d.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()))
    w = np.empty(d.n_params, dtype=np.float32)
    d.get_weights(w)
    n = d.last_step_launches()
    d.destroy()
    return w, losses, n


def test_epilogue_batch_norm_sums_match_separate_reductions():
    """The batch-norm sums taken in the convolution epilogues and the separate reduction kernels are two evaluations
    of the same sums in different orders: six ResNet-20 K=3 bf16 iterations in each mode must end with the same
    weights up to what a last-bit difference of a statistic can move through bf16 rounding, per parameter tensor."""
    wa, la, na = _resnet20_k3_bf16_run()
    wb, lb, nb = _resnet20_k3_bf16_run(separate_bn_sums=True)
    assert nb > na                                                       # the separate reductions are extra launches
    assert np.all(np.isfinite(wa)) and np.all(np.isfinite(wb))
    assert abs(la[-1] - lb[-1]) < 5e-3 * max(1.0, abs(lb[-1]))
    worst = max(rel(wa[off:off + int(np.prod(shape))], wb[off:off + int(np.prod(shape))])
                for _, name, off, shape, _ in nets.param_segments(nets.resnet(3, 10)))
    print("epilogue vs separate sums: worst per-tensor weight difference", worst)
    assert worst < 5e-3


def test_batch_norm_pass_on_the_operand_path_gives_the_same_bits():
    """The normalise + ReLU passes inside the convolution that consumes them (shared memory, between TMA box and MMA;
    fuse_bn_apply = 1: the first batch norm of a block, 2: also the block's closing pass with the shortcut) and the
    separate element-wise kernels compute the same values: identical losses and weights after six iterations, fewer
    launches."""
    wa, la, na = _resnet20_k3_bf16_run()
    wb, lb, nb = _resnet20_k3_bf16_run(fuse_bn_apply=1)
    wc, lc, nc = _resnet20_k3_bf16_run(fuse_bn_apply=2)
    assert nc < nb < na
    assert la == lb == lc and np.array_equal(wa, wb) and np.array_equal(wa, wc)


def test_both_places_of_folding_the_batch_norm_sums_give_the_same_bits():
    """bn_fold = 1 (the convolution's last CTA) and 2 (the consuming element-wise pass) run the same folding routine on
    the same partials: identical losses and weights."""
    wa, la, _ = _resnet20_k3_bf16_run(bn_fold=1)
    wb, lb, _ = _resnet20_k3_bf16_run(bn_fold=2)
    assert la == lb and np.array_equal(wa, wb)


def test_launch_overlap_settings_give_the_same_bits():
    """The programmatic-launch policy only moves kernels in time: never / library policy / every kernel must produce
    identical weights (fixed summation orders everywhere)."""
    ref = _resnet20_k3_bf16_run(launch_overlap=1)[0]
    for mode in (0, 2):
        assert np.array_equal(ref, _resnet20_k3_bf16_run(launch_overlap=mode)[0]), mode


def test_bounded_wait_runs_out_cleanly():
    """A device-side wait that nothing satisfies gives up after its poll limit, the kernel returns, the next sync point
    reports DDG_ERR_TIMEOUT, and from then on the context answers DDG_ERR_STATE; the device stays usable."""
    from paper_1804_10574_b200 import binding
    d = binding.Ddg(nets.mlp(), [1], 4, (64, 1, 1), 10)
    x = torch.zeros(4, 64, device="cuda"); y = torch.zeros(4, dtype=torch.int32, device="cuda")
    d.step(x, y)
    d.debug_wait_timeout(2000)
    with pytest.raises(binding.DdgError) as e:
        d.sync()
    assert e.value.status == 6 and "bounded wait" in str(e.value)
    with pytest.raises(binding.DdgError) as e:
        d.step(x, y)
    assert e.value.status == 7
    d.destroy()
    # another context in the same process starts clean (every context has its own error word)
    d2 = binding.Ddg(nets.mlp(), [1], 4, (64, 1, 1), 10)
    d2.step(x, y)
    d2.sync()
    d2.destroy()
    assert float((torch.ones(8, device="cuda") * 2).sum()) == 16.0


def test_ring_stamps_catch_a_shifted_slot():
    """debug_checks: with the forward counter of module 1 shifted by one, as a ring-indexing error would, the backward
    sweep finds a stamp it does not expect and the next sync point answers DDG_ERR_STATE; unshifted runs stay clean
    (test_graph_replay_over_two_ring_periods_fp32 runs with the stamps on)."""
    from paper_1804_10574_b200 import binding
    L = nets.mlp()
    d = binding.Ddg(L, [0, 1], 4, (64, 1, 1), 10, debug_checks=True, use_graph=True)
    x = torch.zeros(4, 64, device="cuda"); y = torch.zeros(4, dtype=torch.int32, device="cuda")
    for _ in range(5):
        d.step(x, y)
    d.sync()
    d.debug_shift_stamps(0, 1)
    for _ in range(4):
        d.step(x, y, want_loss=False)
    with pytest.raises(binding.DdgError) as e:
        d.sync()
    assert e.value.status == 7 and "ring stamp" in str(e.value)
    d.destroy()


@pytest.mark.parametrize("net,splits,prec", [("resnet8", [1, 2], "bf16"), ("mlp", [1], "fp32")], ids=["resnet8_K3_bf16", "mlp_K2_fp32"])
def test_pipelined_loss_read_back_equals_the_synchronous_run(net, splits, prec):
    """ddg_step_host_pipelined hands out, one call later, exactly the losses ddg_step_host returns (the host runs one
    iteration ahead of the loss it logs); ddg_pipelined_loss returns the last one; the weights after the run are the
    same bits.  Input buffers are reused two calls later, as the contract allows."""
    from paper_1804_10574_b200 import binding, synth
    cfg = nets.config(net)
    B, steps = 8, 14
    kw = dict(precision=prec, lr=0.05, momentum=0.9, weight_decay=5e-4, use_graph=True)
    w0 = synth.init_weights(cfg["layers"], perturb_affine=0.1)
    batches = [synth.batch(t, B, cfg["in_shape"], cfg["num_classes"]) for t in range(steps)]

    a = binding.Ddg(cfg["layers"], splits, B, cfg["in_shape"], cfg["num_classes"], **kw)
    a.set_weights(w0)
    ref = [a.step_host(torch.from_numpy(x).pin_memory(), torch.from_numpy(y).pin_memory()) for x, y in batches]
    wa = a.get_weights(np.empty(a.n_params, dtype=np.float32))
    a.destroy()

    b = binding.Ddg(cfg["layers"], splits, B, cfg["in_shape"], cfg["num_classes"], **kw)
    b.set_weights(w0)
    ring = [(torch.from_numpy(batches[0][0].copy()).pin_memory(), torch.from_numpy(batches[0][1].copy()).pin_memory()) for _ in range(2)]
    got = []
    for t, (x, y) in enumerate(batches):
        xb, yb = ring[t % 2]          # the buffer of iteration t-2: its call for t-1 has returned a loss
        xb.copy_(torch.from_numpy(x)); yb.copy_(torch.from_numpy(y))
        got.append(b.step_host_pipelined(xb, yb))
    last = b.pipelined_loss()
    wb = b.get_weights(np.empty(b.n_params, dtype=np.float32))
    b.destroy()
    assert np.isnan(got[0])
    assert got[1:] == ref[:-1] and last == ref[-1]
    assert np.array_equal(wa, wb)


@pytest.mark.parametrize("graph", [False, True], ids=["eager", "graph"])
def test_piece_times_cover_every_module(graph):
    """time_pieces: every module's forward piece and backward + update piece of the last iteration has a positive device
    time, a module in warm-up (no delayed gradient yet, Eq. 8) spends almost nothing in its backward piece, the pieces
    fit inside the iteration's wall time, and the timed run produces the same weights as the untimed one."""
    import time
    from paper_1804_10574_b200 import binding, synth
    L, B, shape = nets.resnet(1, 10), 32, (3, 32, 32)
    w0 = synth.init_weights(L)
    outs = []
    for timed in (True, False):
        d = binding.Ddg(L, [1, 2], B, shape, 10, precision="bf16", lr=0.01, momentum=0.9, use_graph=graph,
                        time_pieces=timed)
        d.set_weights(w0)
        if not timed:
            with pytest.raises(binding.DdgError) as e:
                d.step(*[torch.from_numpy(a).cuda() for a in synth.batch(0, B, shape, 10)])
                d.piece_times()
            assert e.value.status == 1
            d.destroy()
            d = binding.Ddg(L, [1, 2], B, shape, 10, precision="bf16", lr=0.01, momentum=0.9, use_graph=graph)
            d.set_weights(w0)
        for t in range(8):
            x, y = [torch.from_numpy(a).cuda() for a in synth.batch(t, B, shape, 10)]
            d.sync()
            t0 = time.perf_counter()
            d.step(x, y, want_loss=False)
            d.sync()
            wall_ms = (time.perf_counter() - t0) * 1e3
            if timed:
                f, b = d.piece_times()
                assert len(f) == 3 and len(b) == 3
                assert all(v > 0 for v in f) and all(v >= 0 for v in b), (t, f, b)
                assert max(f + b) < wall_ms + 0.5, (t, f, b, wall_ms)
                if t == 0:      # modules 1 and 2 have no gradient yet: their backward piece is an empty update
                    assert b[0] < 0.25 * b[2] and b[1] < 0.25 * b[2], b
                if t >= 2:
                    assert all(v > 0.01 for v in b), b
        outs.append(d.get_weights(np.empty(d.n_params, dtype=np.float32)))
        d.destroy()
    assert np.array_equal(outs[0], outs[1])


@pytest.mark.parametrize("net,splits,prec,opt", [("resnet8", [1, 2], "bf16", "sgd"), ("mlp", [0, 1, 2], "fp32", "adam"),
                                                  ("resnet8", [2], "fp32", "sgd")], ids=["resnet8_K3_bf16", "mlp_K4_adam", "resnet8_K2_fp32"])
def test_checkpoint_resume_is_exact(net, splits, prec, opt):
    """A checkpoint taken in the middle of a run (modules owe backward sweeps for up to K-1 samples: activation rings,
    weight versions and pending error gradients are part of the state) restored into a fresh context, and restored into
    the context that wrote it, continues bit for bit as the uninterrupted run, graph replay on."""
    from paper_1804_10574_b200 import binding, synth
    cfg = nets.config(net)
    B = 8
    kw = dict(precision=prec, opt=opt, lr=1e-3 if opt == "adam" else 0.05, momentum=0.9, weight_decay=5e-4, use_graph=True)

    def make():
        d = binding.Ddg(cfg["layers"], splits, B, cfg["in_shape"], cfg["num_classes"], **kw)
        d.set_weights(synth.init_weights(cfg["layers"], perturb_affine=0.1))
        return d

    def run(d, t0, t1):
        losses = []
        for t in range(t0, t1):
            x, y = synth.batch(t, B, cfg["in_shape"], cfg["num_classes"])
            losses.append(d.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()))
        w = np.empty(d.n_params, dtype=np.float32)
        d.get_weights(w)
        grads = [np.empty(n, dtype=np.float32) for n in d.per_module]
        samples = [d.get_grads(k, g) for k, g in enumerate(grads)]
        return losses, w, grads, samples

    a = make()
    run(a, 0, 7)
    blob = a.save_state(np.empty(a.state_bytes(), dtype=np.uint8))
    ref = run(a, 7, 12)
    b = make()                       # fresh context: nothing recorded, iteration count 0
    b.load_state(blob)
    got = run(b, 7, 12)
    a.load_state(blob)               # roll the writer back
    again = run(a, 7, 12)
    for other in (got, again):
        assert other[0] == ref[0] and np.array_equal(other[1], ref[1]) and other[3] == ref[3]
        assert all(np.array_equal(g, h) for g, h in zip(other[2], ref[2]))
    c = binding.Ddg(cfg["layers"], splits, B + 1, cfg["in_shape"], cfg["num_classes"], **kw)   # another batch size
    with pytest.raises(binding.DdgError) as e:
        c.load_state(blob)
    assert e.value.status == 1
    for d in (a, b, c):
        d.destroy()
