"""GPU parity of the whole DDG iteration: CUDA library vs CPU oracle, step by step, through the C ABI.
Tolerances: fp32 mode 1e-4 relative per tensor (gradients, weights) and 1e-3 on the loss trajectory; bf16 mode
2e-2 relative against the oracle with the same bf16 storage points."""
import numpy as np
import pytest
import torch

from paper_1804_10574_b200 import nets
from tests.parity import rel, run_pair

pytestmark = pytest.mark.gpu

FP32_TOL, BF16_TOL, LOSS_TOL = 1e-4, 2e-2, 1e-3


def test_mlp_k2_20_steps_fp32():
    w = run_pair(nets.config("mlp"), 20, FP32_TOL, LOSS_TOL)
    print("mlp K=2 worst", w)


@pytest.mark.parametrize("splits", [[], [0], [0, 1, 2]], ids=["K1", "K2_early", "K4"])
def test_mlp_other_splits_fp32(splits):
    run_pair(nets.config("mlp"), 8, FP32_TOL, LOSS_TOL, split_after=splits)


def test_mlp_ragged_batch_and_momentum_fp32():
    cfg = dict(nets.config("mlp"), opt=dict(lr=0.05, momentum=0.9, weight_decay=1e-3))
    run_pair(cfg, 8, FP32_TOL, LOSS_TOL, batch=7)


def test_mlp_adam_fp32():
    cfg = dict(nets.config("mlp"), opt=dict(lr=1e-3, momentum=0.0, weight_decay=0.0))
    run_pair(cfg, 8, FP32_TOL, LOSS_TOL, opt="adam")


def test_mlp_diminishing_stepsize_fp32():
    run_pair(nets.config("mlp"), 6, FP32_TOL, LOSS_TOL, lr_schedule=lambda t: 0.05 / (1 + t))


def test_resnet8_k2_20_steps_fp32():
    w = run_pair(nets.config("resnet8"), 20, FP32_TOL, LOSS_TOL)
    print("resnet8 K=2 worst", w)


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
    run_pair(cfg, 5, BF16_TOL, 5e-3, precision="bf16", split_after=split, noise_mult=2.0)


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
    w = run_pair(cfg, 6, BF16_TOL, 5e-3, precision="bf16", noise_mult=2.0)
    print("resnet8 bf16 worst", w)


def test_resnet20_k3_bf16_graph():
    L = nets.resnet(3, 10)
    cfg = dict(layers=L, split_after=nets.split_even_blocks(L, 3), batch=32, in_shape=(3, 32, 32), num_classes=10,
               precision="bf16", opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    w = run_pair(cfg, 8, BF16_TOL, 5e-3, use_graph=True, noise_mult=2.0)
    print("resnet20 bf16 worst", w)


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
    w = run_pair(cfg, 5, BF16_TOL, 5e-3, use_graph=True, noise_mult=2.0, check_every=2)
    print("resnet110 K=4 full size worst", w)


_CHILD = r"""
import sys, numpy as np, torch
from paper_1804_10574_b200 import binding, nets, synth
L = nets.resnet(3, 10)
B, shape, classes = 32, (3, 32, 32), 10
d = binding.Ddg(L, nets.split_even_blocks(L, 3), B, shape, classes, precision="bf16", lr=0.01, momentum=0.9,
                weight_decay=5e-4, use_graph=True)
d.set_weights(synth.init_weights(L, perturb_affine=0.1))
losses = []
for t in range(6):
    x, y = synth.batch(t, B, shape, classes)
    losses.append(d.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()))
w = np.empty(d.n_params, dtype=np.float32)
d.get_weights(w)
np.save(sys.argv[1], np.concatenate([w, np.asarray(losses, dtype=np.float32)]))
"""


def test_epilogue_batch_norm_sums_match_separate_reductions(tmp_path):
    """The batch-norm sums taken in the convolution epilogues and the separate reduction kernels are two evaluations
    of the same sums in different orders: six ResNet-20 K=3 bf16 iterations in each mode (the switch is read once per
    process, so each runs in a child) must end with the same weights up to what a last-bit difference of a statistic
    can move through bf16 rounding."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = {}
    for mode in ("1", "0"):
        f = str(tmp_path / ("w%s.npy" % mode))
        env = dict(os.environ, DDG_FUSE_BN=mode, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
        subprocess.run([sys.executable, "-c", _CHILD, f], check=True, env=env, cwd=root, timeout=600)
        out[mode] = np.load(f)
    a, b = out["1"], out["0"]
    assert np.all(np.isfinite(a)) and np.all(np.isfinite(b))
    assert abs(a[-1] - b[-1]) < 5e-3 * max(1.0, abs(b[-1]))          # last loss
    assert rel(a[:-6], b[:-6]) < 2e-3                                  # all weights, one tensor

