"""Pins for the oracle's DDG iteration (Section 3.1 Eq. 6-7, Section 3.3 Eq. 8-9, Algorithms 1-2) against
what the paper fixes: K=1 is plain backprop, delays are K-1..0, the delayed gradient is the true gradient of the
stored iteration at the stored weights, warm-up gradients are zero, and the update rule.  No GPU."""
import numpy as np
import pytest
import torch

from oracle import ddg_oracle as orc
from paper_1804_10574_b200 import nets, synth
from tests import torch_bp

TINY_RESNET = dict(layers=nets.resnet(1, 5, channels=(4, 4, 8, 8)), in_shape=(3, 8, 8), num_classes=5, batch=4)
TINY_RESNET_PROJ = dict(layers=nets.resnet(1, 5, channels=(4, 4, 8, 8), projection=True), in_shape=(3, 8, 8), num_classes=5, batch=4)
TINY_MLP = dict(layers=nets.mlp((6, 8, 8, 7, 5)), in_shape=(6, 1, 1), num_classes=5, batch=4)


def make(net, split_after, **kw):
    o = orc.Oracle(net["layers"], split_after, net["batch"], net["in_shape"], net["num_classes"], **kw)
    w0 = synth.init_weights(net["layers"], perturb_affine=0.1).astype(np.float64)
    o.set_weights(w0)
    return o, w0


def data(net, t):
    return synth.batch(t, net["batch"], net["in_shape"], net["num_classes"])


def rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def module_slices(o):
    off, out = 0, []
    for n in o.per_module:
        out.append(slice(off, off + n))
        off += n
    return out


@pytest.mark.parametrize("net", [TINY_MLP, TINY_RESNET, TINY_RESNET_PROJ], ids=["mlp", "resnet", "resnet_proj"])
def test_whole_net_finite_differences(net):
    """Every layer's backward sweep, chained: the K=1 gradient equals central differences of the loss."""
    o, w0 = make(net, [], lr=0.0)
    x, y = data(net, 0)
    o.step(x, y)
    _, g = o.get_grads(0)
    rng = np.random.default_rng(3)
    idx = rng.choice(w0.size, size=min(w0.size, 120), replace=False)
    h = 1e-6
    for i in idx:
        w = w0.copy(); w[i] += h; o.set_weights(w); fp = o.loss_only(x, y)
        w[i] -= 2 * h; o.set_weights(w); fm = o.loss_only(x, y)
        assert abs((fp - fm) / (2 * h) - g[i]) < 1e-6 * max(1.0, abs(g[i])), i


@pytest.mark.parametrize("net", [TINY_MLP, TINY_RESNET, TINY_RESNET_PROJ], ids=["mlp", "resnet", "resnet_proj"])
def test_k1_is_plain_backprop_with_sgd(net):
    """Section 3.2: with K=1 there is no delay and DDG is backpropagation + SGD (Eq. 2), step by step."""
    lr = 0.05
    o, w0 = make(net, [], lr=lr)
    w = w0.copy()
    for t in range(4):
        x, y = data(net, t)
        loss_ref, g_ref = torch_bp.loss_and_grad(net["layers"], w, x, y)
        loss = o.step(x, y)
        s, g = o.get_grads(0)
        assert s == t and abs(loss - loss_ref) < 1e-12
        assert rel(g, g_ref) < 1e-10
        w = w - lr * g_ref
        assert rel(o.get_weights(), w) < 1e-11


@pytest.mark.parametrize("K,splits,net", [(2, [2], TINY_RESNET), (3, [2, 3], TINY_RESNET), (4, [1, 2, 3], TINY_RESNET),
                                          (3, [2, 3], TINY_RESNET_PROJ)], ids=["K2", "K3", "K4", "K3_proj"])
def test_delayed_gradient_is_true_gradient_of_stored_iteration(K, splits, net):
    """Eq. 8-9: g_k applied at iteration t is [grad f_{x_s}(w^s)]_{G(k)} with s = t-K+k; delays run from K-1
    (k=1) to 0 (k=K); zero during warm-up, when the module's weights must not move (plain SGD)."""
    lr = 0.05
    o, w0 = make(net, splits, lr=lr)
    sl = module_slices(o)
    snapshots, batches = [], []
    for t in range(K + 4):
        x, y = data(net, t)
        snapshots.append(o.get_weights())
        batches.append((x, y))
        before = o.get_weights()
        loss = o.step(x, y)
        after = o.get_weights()
        loss_ref, _ = torch_bp.loss_and_grad(net["layers"], snapshots[t], x, y)
        assert abs(loss - loss_ref) < 1e-11
        for k in range(1, K + 1):
            s, g = o.get_grads(k - 1)
            if t - K + k < 0:
                assert s == -1 and not g.any()
                np.testing.assert_array_equal(after[sl[k - 1]], w0[sl[k - 1]])   # bit-identical to init
                continue
            assert s == t - K + k                                               # delay K-k
            _, g_ref = torch_bp.loss_and_grad(net["layers"], snapshots[s], *batches[s])
            assert rel(g, g_ref[sl[k - 1]]) < 1e-9, (t, k)
            np.testing.assert_allclose(after[sl[k - 1]] - before[sl[k - 1]], -lr * g, rtol=1e-9, atol=1e-15)


def test_k3_module_A_uses_delta_two_iterations_old():
    """Figure 2: with three modules, module A (k=1) runs on the error gradient of iteration t-2."""
    o, _ = make(TINY_MLP, [0, 2], lr=0.01)
    seen = []
    for t in range(5):
        o.step(*data(TINY_MLP, t))
        seen.append([o.get_grads(k)[0] for k in range(3)])
    assert seen == [[-1, -1, 0], [-1, 0, 1], [0, 1, 2], [1, 2, 3], [2, 3, 4]]


def test_lr_zero_keeps_weights_and_makes_ddg_grads_bp_grads():
    net = TINY_RESNET
    o, w0 = make(net, [2, 3], lr=0.0, momentum=0.9)
    sl = module_slices(o)
    bs = []
    for t in range(5):
        bs.append(data(net, t))
        o.step(*bs[t])
        np.testing.assert_array_equal(o.get_weights(), w0)
        for k in range(3):
            s, g = o.get_grads(k)
            if s >= 0:
                _, g_ref = torch_bp.loss_and_grad(net["layers"], w0, *bs[s])
                assert rel(g, g_ref[sl[k]]) < 1e-9


def test_stored_weights_versus_current_weights_reading():
    """Eq. 6-7 differentiate at w^{t-K+k}.  The alternative reading (current weights) gives a different
    gradient for the lower module as soon as the weights have moved, and the same one while lr = 0."""
    net = TINY_RESNET
    a, _ = make(net, [2], lr=0.1)
    b, _ = make(net, [2], lr=0.1, flags=orc.USE_CURRENT_WEIGHTS)
    for t in range(3):
        a.step(*data(net, t)); b.step(*data(net, t))
    assert rel(a.get_grads(0)[1], b.get_grads(0)[1]) > 1e-6
    a, _ = make(net, [2], lr=0.0)
    b, _ = make(net, [2], lr=0.0, flags=orc.USE_CURRENT_WEIGHTS)
    for t in range(3):
        a.step(*data(net, t)); b.step(*data(net, t))
    np.testing.assert_array_equal(a.get_grads(0)[1], b.get_grads(0)[1])


def test_momentum_weight_decay_matches_library_optimiser_at_k1():
    """With K=1 the update d = g + wd*w, v = mu*v + d, w -= lr*v is the library's SGD(momentum, weight_decay)."""
    net = TINY_MLP
    lr, mu, wd = 0.1, 0.9, 5e-4
    o, w0 = make(net, [], lr=lr, momentum=mu, weight_decay=wd)
    wt = torch.tensor(w0.copy(), requires_grad=True)
    opt = torch.optim.SGD([wt], lr=lr, momentum=mu, weight_decay=wd)
    for t in range(5):
        x, y = data(net, t)
        opt.zero_grad()
        torch_bp.forward(net["layers"], wt, torch.tensor(x, dtype=torch.float64), torch.tensor(y).long()).backward()
        opt.step()
        o.step(x, y)
        assert rel(o.get_weights(), wt.detach().numpy()) < 1e-11


def test_warmup_rule_and_its_literal_alternative():
    net = TINY_MLP
    o, w0 = make(net, [1], lr=0.1, momentum=0.9, weight_decay=0.1)
    o.step(*data(net, 0))
    n0 = o.per_module[0]
    np.testing.assert_array_equal(o.get_weights()[:n0], w0[:n0])           # no update at all while s < 0
    o2, _ = make(net, [1], lr=0.1, momentum=0.9, weight_decay=0.1, flags=orc.WARMUP_DECAY)
    o2.step(*data(net, 0))
    np.testing.assert_allclose(o2.get_weights()[:n0], w0[:n0] * (1 - 0.1 * 0.1), rtol=1e-14)  # g=0: decay only


def test_adam_ddg_matches_library_adam_at_k1_and_is_still_during_warmup():
    """Algorithm 2: eps 1e-8, betas (0.9, 0.999), bias correction with the global t+1."""
    net = TINY_MLP
    o, w0 = make(net, [], opt="adam", lr=1e-3)
    wt = torch.tensor(w0.copy(), requires_grad=True)
    opt = torch.optim.Adam([wt], lr=1e-3, betas=(0.9, 0.999), eps=1e-8)
    for t in range(5):
        x, y = data(net, t)
        opt.zero_grad()
        torch_bp.forward(net["layers"], wt, torch.tensor(x, dtype=torch.float64), torch.tensor(y).long()).backward()
        opt.step()
        o.step(x, y)
        assert rel(o.get_weights(), wt.detach().numpy()) < 1e-9
    # K=2: module 1 has zero gradient at t=0, so m=v=0 and the Adam step is exactly zero
    o, w0 = make(net, [1], opt="adam", lr=1e-3)
    o.step(*data(net, 0))
    n0 = o.per_module[0]
    np.testing.assert_array_equal(o.get_weights()[:n0], w0[:n0])
    # at t=1 module 1 takes its first real Adam step with bias correction 1-beta^2 (global t+1 = 2), not 1-beta
    o.step(*data(net, 1))
    _, g = o.get_grads(0)
    m, v = 0.1 * g, 0.001 * g * g
    expect = w0[:n0] - 1e-3 * (m / (1 - 0.9 ** 2)) / (np.sqrt(v / (1 - 0.999 ** 2)) + 1e-8)
    np.testing.assert_allclose(o.get_weights()[:n0], expect, rtol=1e-10, atol=1e-14)


def test_param_counts_match_table_2():
    from tests.test_oracle_layers import golden
    g = golden()
    for classes, key in ((100, "resnet110_params_100"), (10, "resnet110_params_10")):
        L = nets.resnet(18, classes)
        o = orc.Oracle(L, nets.split_even_blocks(L, 4), 1, (3, 32, 32), classes)
        assert o.n_params == int(g[key]) == nets.param_count(L)
        assert len(o.per_module) == 4
    L = nets.resnet(18, 100)
    assert nets.split_even_blocks(L, 4) == [15, 29, 42]          # 14, 14, 13, 13 blocks
    assert nets.split_even_blocks(nets.resnet(9, 10), 2) == [15]  # 14 + 13 blocks


def test_bf16_rounding_switch_perturbs_but_does_not_change_the_method():
    """Storage rounding is a perturbation of the evaluation point: the loss barely moves; gradients move by a
    few percent (they are small differences of large terms), and every DDG index stays the same."""
    net = dict(layers=nets.resnet(1, 10), in_shape=(3, 32, 32), num_classes=10, batch=8)
    a, _ = make(net, [2], lr=0.0)
    b, _ = make(net, [2], lr=0.0, flags=orc.ROUND_BF16)
    for t in range(2):
        la, lb = a.step(*data(net, t)), b.step(*data(net, t))
        assert abs(la - lb) < 1e-2
        for k in range(2):
            (sa, ga), (sb, gb) = a.get_grads(k), b.get_grads(k)
            assert sa == sb
            if sa >= 0:
                assert 1e-5 < rel(gb, ga) < 0.3


def test_fp32_storage_rounding_is_a_tiny_perturbation_of_the_exact_run():
    """ORC_ROUND_FP32 only rounds what is stored: the run must stay within float rounding of the exact one."""
    net = dict(layers=nets.resnet(1, 10), in_shape=(3, 16, 16), num_classes=10, batch=4)
    a, _ = make(net, [2], lr=0.05, momentum=0.9, weight_decay=5e-4)
    b, _ = make(net, [2], lr=0.05, momentum=0.9, weight_decay=5e-4, flags=orc.ROUND_FP32)
    for t in range(3):
        la, lb = a.step(*data(net, t)), b.step(*data(net, t))
        assert abs(la - lb) < 1e-5
    assert rel(b.get_weights(), a.get_weights()) < 1e-5
    w = b.get_weights()
    np.testing.assert_array_equal(w, w.astype(np.float32).astype(np.float64))   # master weights are float values
    sb, gb = b.get_grads(1)
    np.testing.assert_array_equal(gb, gb.astype(np.float32).astype(np.float64))
