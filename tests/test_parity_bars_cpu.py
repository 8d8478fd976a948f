"""What the bf16 acceptance rule of tests/parity.py lets through and what it rejects, shown on the CPU with the
oracle alone (no GPU, no CUDA path involved).

The rule compares a candidate gradient with the oracle's bf16-storage run and with its exact run.  A correct
evaluation that merely rounds differently must pass; a zero gradient, a gradient of another sample (a stale ring
slot), a scaled or a sign-flipped gradient must fail, also when the format noise is as large as the gradient itself
(deep networks), where a bound on the distance alone would accept all of them."""
import numpy as np
import pytest

from oracle import ddg_oracle as orc
from paper_1804_10574_b200 import nets, synth
from tests.parity import (MODULE_DIR_KEEP, MODULE_DIR_SLACK, bf16_tensor_verdict, module_direction,
                          segments_by_module)

TOL = 2e-2


def _grads(flags, w0, layers, splits, B, shape, steps, scale_w=None):
    o = orc.Oracle(layers, splits, B, shape, 10, lr=0.01, momentum=0.9, weight_decay=5e-4, flags=flags)
    w = w0.astype(np.float64)
    if scale_w is not None:
        w = w * scale_w
    o.set_weights(w)
    out = []
    for t in range(steps):
        o.step(*synth.batch(t, B, shape, 10))
        out.append([o.get_grads(k) for k in range(len(splits) + 1)])
    o.close()
    return out


def test_bar_on_oracle_gradients_of_a_small_resnet():
    layers, splits, B, shape, steps = nets.resnet(1, 10), [2], 8, (3, 16, 16), 4
    w0 = synth.init_weights(layers, perturb_affine=0.1)
    exact = _grads(0, w0, layers, splits, B, shape, steps)
    bf16 = _grads(orc.ROUND_BF16, w0, layers, splits, B, shape, steps)
    # the same problem evaluated with weights that differ by 1e-7 relative (about what fp32 accumulation differs from
    # fp64 by): its bf16 rounding decisions drift apart from the first run's - a correct, differently rounded path
    jitter = 1.0 + 1e-7 * np.random.default_rng(1).standard_normal(w0.size)
    other = _grads(orc.ROUND_BF16, w0, layers, splits, B, shape, steps, scale_w=jitter)
    segs = segments_by_module(layers, splits)
    checked = rejected_stale = 0
    for t in range(1, steps):
        for k in range(2):
            s, g_ex = exact[t][k]
            if s < 1:
                continue
            g_bf, g_ok = bf16[t][k][1], other[t][k][1]
            g_stale = bf16[t - 1][k][1]                       # the gradient of the previous sample
            c_orc = module_direction(g_bf, g_ex, segs[k])
            assert module_direction(g_ok, g_ex, segs[k]) >= MODULE_DIR_KEEP * c_orc - MODULE_DIR_SLACK
            assert module_direction(g_stale, g_ex, segs[k]) < MODULE_DIR_KEEP * c_orc - MODULE_DIR_SLACK
            assert module_direction(np.zeros_like(g_ex), g_ex, segs[k]) < MODULE_DIR_KEEP * c_orc - MODULE_DIR_SLACK
            for name, a, b in segs[k]:
                ok, why, _ = bf16_tensor_verdict(g_ok[a:b], g_bf[a:b], g_ex[a:b], TOL)
                assert ok, (t, k, name, why)
                assert not bf16_tensor_verdict(np.zeros(b - a), g_bf[a:b], g_ex[a:b], TOL)[0], (t, k, name, "zero")
                assert not bf16_tensor_verdict(2.0 * g_bf[a:b], g_bf[a:b], g_ex[a:b], TOL)[0], (t, k, name, "doubled")
                assert not bf16_tensor_verdict(-g_bf[a:b], g_bf[a:b], g_ex[a:b], TOL)[0], (t, k, name, "sign")
                checked += 1
                rejected_stale += not bf16_tensor_verdict(g_stale[a:b], g_bf[a:b], g_ex[a:b], TOL)[0]
    assert checked >= 20
    assert rejected_stale == checked          # every tensor of a stale-sample gradient is rejected


@pytest.mark.parametrize("noise", [0.3, 1.05])
def test_bar_when_the_format_noise_is_as_large_as_the_gradient(noise):
    """Synthetic vectors with the statistics of the deep case (noise / signal about 1): candidate = exact + independent
    noise passes; zero, stale (another sample's exact + noise), doubled and flipped candidates fail, although the
    distance rule alone (2 x noise + tol) would accept the zero and the stale one at noise 1.05."""
    rng = np.random.default_rng(7)
    n = 9216
    unit = lambda: rng.standard_normal(n) / np.sqrt(n)
    g_ex, g_ex2 = unit(), unit()
    g_bf = g_ex + noise * unit()
    good = g_ex + noise * unit()
    stale = g_ex2 + noise * unit()
    assert bf16_tensor_verdict(good, g_bf, g_ex, TOL)[0]
    for name, cand in (("zero", np.zeros(n)), ("stale", stale), ("doubled", 2 * good), ("flipped", -good)):
        ok, why, _ = bf16_tensor_verdict(cand, g_bf, g_ex, TOL)
        assert not ok, (name, why)
    if noise > 1.0:   # what a distance-only rule would have said
        from tests.parity import NOISE_MULT, rel
        assert rel(np.zeros(n), g_ex) <= NOISE_MULT * rel(g_bf, g_ex) + TOL
        assert rel(stale, g_ex) <= NOISE_MULT * rel(g_bf, g_ex) + TOL
