"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle side by side on the same
seeded inputs and compare loss, delayed gradients and weights per tensor.

The acceptance rules are plain functions of arrays (no GPU needed), so that the CPU test suite can show what they
reject: see tests/test_parity_bars_cpu.py."""
import numpy as np

from oracle import ddg_oracle as orc
from paper_1804_10574_b200 import nets, synth


def rel(a, b):
    """Per-tensor relative error: ||a-b||_2 / max(||b||_2, 1e-12)."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-12))


def cosine(a, b):
    a, b = np.asarray(a, dtype=np.float64).ravel(), np.asarray(b, dtype=np.float64).ravel()
    return float(a @ b / max(np.linalg.norm(a) * np.linalg.norm(b), 1e-300))


def elementwise_ok(got, ref, rtol, atol):
    """|got - ref| <= rtol * |ref| + atol for every element; returns (ok, index of the worst element, its excess)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    excess = np.abs(got - ref) - (rtol * np.abs(ref) + atol)
    i = int(np.argmax(excess))
    return bool(excess.flat[i] <= 0.0), np.unravel_index(i, excess.shape), float(excess.flat[i])


def segments_by_module(layers, split_after):
    """{module: [(name, start, stop)]} with offsets relative to the module's parameter slice."""
    bounds = [-1] + list(split_after) + [len(layers) - 1]
    segs = nets.param_segments(layers)
    sizes = {(i, name): int(np.prod(shape)) for i, name, off, shape, _ in segs}
    out = {}
    for k in range(len(bounds) - 1):
        mine = [(i, name, off) for i, name, off, shape, _ in segs if bounds[k] < i <= bounds[k + 1]]
        base = mine[0][2] if mine else 0
        out[k] = [("L%d.%s" % (i, name), off - base, off - base + sizes[(i, name)]) for i, name, off in mine]
    return out


# ---- the bf16 bar ------------------------------------------------------------------------------------------
# Rounding every stored tensor to bf16 makes two evaluations that differ in the last bit before a store decorrelate
# within a few layers (a one-ulp difference of one activation flips the rounding of a share of the next layer's
# outputs), so a path that accumulates in fp32 cannot reproduce the oracle's bf16 decisions: its gradients carry an
# independent draw of the same format noise.  The oracle measures that noise itself: with g_exact from the exact run
# and g_bf16 from the run with bf16 storage, e_orc = rel(g_bf16, g_exact).  A gradient tensor g passes when it is
# within `tol` of g_bf16, or when ALL of the following hold:
#   size      rel(g, g_exact) <= NOISE_MULT * e_orc + tol          (its noise is no larger than the format's own)
#   length    ||g|| / ||g_bf16|| in [1/LEN_BAND, LEN_BAND]          (noise is independent of the signal: same length)
#   direction cos(g, g_exact) >= DIR_KEEP * cos(g_bf16, g_exact) - DIR_SLACK   (tensors of >= DIR_MIN_ELEMS values)
# The size rule alone lets a zero or stale gradient through once e_orc approaches 1 (deep networks); the length rule
# rejects zero and scaled gradients, the direction rule rejects gradients of another sample or ring slot.
NOISE_MULT, LEN_BAND, DIR_KEEP, DIR_SLACK, DIR_MIN_ELEMS = 2.0, 1.6, 0.7, 0.05, 1024


def bf16_tensor_verdict(g, g_bf16, g_exact, tol):
    """(ok, reason, stats) of one gradient (or weight) tensor under the bf16 bar above."""
    g, g_bf16, g_exact = (np.asarray(a, dtype=np.float64).ravel() for a in (g, g_bf16, g_exact))
    e_ref = rel(g, g_bf16)
    e, e_orc = rel(g, g_exact), rel(g_bf16, g_exact)
    st = dict(e_ref=e_ref, e=e, e_orc=e_orc)
    if e_ref <= tol:
        return True, "within tol of the bf16-storage oracle", st
    if e > NOISE_MULT * e_orc + tol:
        return False, "size: %.3e from the exact oracle, format noise %.3e" % (e, e_orc), st
    ratio = np.linalg.norm(g) / max(np.linalg.norm(g_bf16), 1e-300)
    st["len_ratio"] = float(ratio)
    if not (1.0 / LEN_BAND <= ratio <= LEN_BAND):
        return False, "length: ||g|| / ||g_bf16|| = %.3f" % ratio, st
    if g.size >= DIR_MIN_ELEMS:
        c, c_orc = cosine(g, g_exact), cosine(g_bf16, g_exact)
        st["cos"], st["cos_orc"] = c, c_orc
        if c < DIR_KEEP * c_orc - DIR_SLACK:
            return False, "direction: cos %.3f against the exact gradient, the oracle's own bf16 run keeps %.3f" % (c, c_orc), st
    return True, "format noise", st


def module_direction(g, g_exact, segs):
    """cos between two module gradients with every tensor scaled to unit exact norm (all tensors weigh the same)."""
    a = np.concatenate([np.asarray(g[lo:hi], dtype=np.float64) / max(np.linalg.norm(g_exact[lo:hi]), 1e-300) for _, lo, hi in segs])
    b = np.concatenate([np.asarray(g_exact[lo:hi], dtype=np.float64) / max(np.linalg.norm(g_exact[lo:hi]), 1e-300) for _, lo, hi in segs])
    return cosine(a, b)


MODULE_DIR_KEEP, MODULE_DIR_SLACK = 0.9, 0.02


def run_pair(cfg, steps, tol, loss_tol, precision=None, split_after=None, use_graph=False, opt="sgd",
             perturb_affine=0.1, batch=None, check_every=1, lr_schedule=None, noise_bar=False, exact_too=False,
             ratio_band=None, gpu_kwargs=None, exact_loss_tol=None):
    """Step both implementations `steps` times; assert parity at every `check_every`-th step.  Returns the worst
    relative errors seen, for reporting.

    noise_bar (bf16 production kernels): gradients and weights are held to bf16_tensor_verdict and, per module, to
    the direction rule on the whole module gradient; ratio_band = (lo, hi) additionally bounds the median over all
    checked gradient tensors of rel(gpu, exact) / rel(oracle_bf16, exact): an independent draw of the same noise gives
    about 1, a systematic error does not.
    exact_too (fp32 mode): the run is also compared with the exact oracle (no storage rounding at all); the worst
    errors are returned under *_vs_exact and the loss is held to exact_loss_tol (default loss_tol) against it."""
    import torch
    from paper_1804_10574_b200 import binding
    layers = cfg["layers"]
    split_after = cfg["split_after"] if split_after is None else split_after
    precision = precision or cfg["precision"]
    B = batch or cfg["batch"]
    K = len(split_after) + 1
    o = cfg["opt"]
    # the oracle imitates the storage formats of the mode under test (all its arithmetic stays fp64) and gets
    # the hyper-parameters as the float32 values the C ABI carries
    flags = orc.ROUND_BF16 if precision == "bf16" else orc.ROUND_FP32
    f32 = lambda v: float(np.float32(v))
    o = dict(lr=f32(o["lr"]), momentum=f32(o["momentum"]), weight_decay=f32(o["weight_decay"]))

    def oracle(fl):
        r = orc.Oracle(layers, split_after, B, cfg["in_shape"], cfg["num_classes"], opt=opt, lr=o["lr"],
                       momentum=o["momentum"], weight_decay=o["weight_decay"], beta1=f32(0.9), beta2=f32(0.999),
                       eps=f32(1e-8), flags=fl)
        r.set_weights(w0.astype(np.float64))
        return r

    w0 = synth.init_weights(layers, perturb_affine=perturb_affine)
    ref = oracle(flags)
    exact = oracle(0) if (noise_bar or exact_too) else None
    gpu = binding.Ddg(layers, split_after, B, cfg["in_shape"], cfg["num_classes"], precision=precision, opt=opt,
                      lr=o["lr"], momentum=o["momentum"], weight_decay=o["weight_decay"], use_graph=use_graph,
                      **(gpu_kwargs or {}))
    gpu.set_weights(w0)
    assert gpu.n_params == ref.n_params and gpu.per_module == ref.per_module
    segs = segments_by_module(layers, split_after)
    worst = dict(loss=0.0, grad=0.0, weight=0.0, grad_vs_exact=0.0, weight_vs_exact=0.0, loss_vs_exact=0.0,
                 oracle_vs_exact=0.0, ratios=[], min_cos_margin=1.0)
    wbuf = np.empty(gpu.n_params, dtype=np.float32)
    for t in range(steps):
        if lr_schedule is not None:
            ref.set_lr(f32(lr_schedule(t))); gpu.set_lr(lr_schedule(t))
            if exact is not None:
                exact.set_lr(f32(lr_schedule(t)))
        x, y = synth.batch(t, B, cfg["in_shape"], cfg["num_classes"])
        xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
        loss_gpu = gpu.step(xd, yd)
        loss_ref = ref.step(x, y)
        loss_ex = exact.step(x, y) if exact is not None else None
        if t % check_every and t != steps - 1:
            continue
        dl = abs(loss_gpu - loss_ref) / max(1.0, abs(loss_ref))
        worst["loss"] = max(worst["loss"], dl)
        assert dl <= loss_tol, "step %d: loss %r vs oracle %r" % (t, loss_gpu, loss_ref)
        if exact_too:
            dle = abs(loss_gpu - loss_ex) / max(1.0, abs(loss_ex))
            worst["loss_vs_exact"] = max(worst["loss_vs_exact"], dle)
            assert dle <= (exact_loss_tol or loss_tol), "step %d: loss %r vs exact oracle %r" % (t, loss_gpu, loss_ex)
        off = 0
        gpu.get_weights(wbuf)
        wref = ref.get_weights()
        w_ex = exact.get_weights() if exact is not None else None
        for k in range(K):
            gbuf = np.empty(gpu.per_module[k], dtype=np.float32)
            s_gpu = gpu.get_grads(k, gbuf)
            s_ref, g_ref = ref.get_grads(k)
            assert s_gpu == s_ref == (t - K + k + 1 if t - K + k + 1 >= 0 else -1), (t, k, s_gpu, s_ref)
            g_ex = exact.get_grads(k)[1] if exact is not None else None
            if noise_bar and s_ref >= 0:
                c_gpu, c_orc = module_direction(gbuf, g_ex, segs[k]), module_direction(g_ref, g_ex, segs[k])
                worst["min_cos_margin"] = min(worst["min_cos_margin"], c_gpu - MODULE_DIR_KEEP * c_orc)
                assert c_gpu >= MODULE_DIR_KEEP * c_orc - MODULE_DIR_SLACK, \
                    "step %d module %d: direction of the whole gradient %.3f, the oracle's bf16 run keeps %.3f" % (t, k, c_gpu, c_orc)
            for name, a, b in segs[k]:
                if s_ref < 0:
                    assert not gbuf[a:b].any()
                elif noise_bar:
                    ok, why, st = bf16_tensor_verdict(gbuf[a:b], g_ref[a:b], g_ex[a:b], tol)
                    worst["grad"] = max(worst["grad"], st["e_ref"])
                    worst["grad_vs_exact"] = max(worst["grad_vs_exact"], st["e"])
                    worst["oracle_vs_exact"] = max(worst["oracle_vs_exact"], st["e_orc"])
                    if st["e_orc"] > 0:
                        worst["ratios"].append(st["e"] / st["e_orc"])
                    assert ok, "step %d module %d grad %s: %s" % (t, k, name, why)
                else:
                    e = rel(gbuf[a:b], g_ref[a:b])
                    worst["grad"] = max(worst["grad"], e)
                    assert e <= tol, "step %d module %d grad %s: rel %.3e > %.1e" % (t, k, name, e, tol)
                    if exact_too:
                        worst["grad_vs_exact"] = max(worst["grad_vs_exact"], rel(gbuf[a:b], g_ex[a:b]))
                wg, wr = wbuf[off + a:off + b], wref[off + a:off + b]
                e = rel(wg, wr)
                worst["weight"] = max(worst["weight"], e)
                if noise_bar:
                    # weights integrate the gradients, so they carry the same format noise: same size rule
                    ew, ew_orc = rel(wg, w_ex[off + a:off + b]), rel(wr, w_ex[off + a:off + b])
                    assert e <= tol or ew <= NOISE_MULT * ew_orc + tol, \
                        "step %d module %d weight %s: rel %.3e > %.1e (format noise %.3e)" % (t, k, name, e, tol, ew_orc)
                else:
                    assert e <= tol, "step %d module %d weight %s: rel %.3e > %.1e" % (t, k, name, e, tol)
                    if exact_too:
                        worst["weight_vs_exact"] = max(worst["weight_vs_exact"], rel(wg, w_ex[off + a:off + b]))
            off += gpu.per_module[k]
    gpu.destroy()
    ref.close()
    if exact is not None:
        exact.close()
    if worst["ratios"]:
        r = np.asarray(worst["ratios"])
        worst["ratio_median"], worst["ratio_max"] = float(np.median(r)), float(r.max())
        if ratio_band is not None:
            assert ratio_band[0] <= worst["ratio_median"] <= ratio_band[1], \
                "median of rel(gpu, exact) / rel(oracle_bf16, exact) = %.3f outside %r" % (worst["ratio_median"], ratio_band)
    del worst["ratios"]
    return worst
