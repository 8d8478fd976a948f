"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle side by side on the same
seeded inputs and compare loss, delayed gradients and weights per tensor."""
import numpy as np
import torch

from oracle import ddg_oracle as orc
from paper_1804_10574_b200 import nets, synth


def rel(a, b):
    """Per-tensor relative error: ||a-b||_2 / max(||b||_2, 1e-12)."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-12))


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


class TieExplainer:
    """ReLU decisions that floating point cannot settle.

    relu'(z) jumps at z = 0, so two correct evaluations of the same network (fp64 on the CPU, fp32 sums in another
    order on the GPU) may disagree on the derivative of the few elements whose pre-activation is within rounding
    distance of zero, and each such element moves these small, cancellation-dominated gradients by up to a percent.
    The backward sweep is linear in each of those 0/1 decisions, so every valid result has the form
    g = g_off + sum_i c_i * (g_i - g_off) with c_i in {0, 1}, where g_off forces all near-zero decisions off and g_i
    switches only the i-th one on.  The oracle computes g_off and the g_i (plain backprop at the snapshot w^s, which
    the delayed gradient equals by Eq. 8); the GPU gradient must match one member of that family to the strict
    tolerance."""

    def __init__(self, cfg, B, flags, tau=2e-5, max_ties=200):
        self.cfg, self.B, self.flags, self.tau, self.max_ties = cfg, B, flags, tau, max_ties
        self.cache = {}

    def family(self, s, w_snapshot, x, y):
        if s in self.cache:
            return self.cache[s]
        cfg = self.cfg
        o = orc.Oracle(cfg["layers"], [], self.B, cfg["in_shape"], cfg["num_classes"], lr=0.0, flags=self.flags)
        o.set_weights(w_snapshot)
        o.set_tie_policy(self.tau, -1)
        o.step(x, y)
        n = o.tie_count()
        g_off = o.get_grads(0)[1]
        deltas = []
        if n <= self.max_ties:
            for i in range(n):
                o.set_tie_policy(self.tau, i)
                o.step(x, y)
                deltas.append(o.get_grads(0)[1] - g_off)
        o.close()
        self.cache[s] = (g_off, deltas, n)
        return self.cache[s]

    def residual(self, s, w_snapshot, x, y, lo, hi, g_gpu):
        """Best member of the family on the parameter range [lo, hi): returns (residual vector, coefficients)."""
        g_off, deltas, n = self.family(s, w_snapshot, x, y)
        b = np.asarray(g_gpu, dtype=np.float64) - g_off[lo:hi]
        if not deltas:
            return b, np.zeros(0), n
        A = np.stack([d[lo:hi] for d in deltas], axis=1)
        keep = np.linalg.norm(A, axis=0) > 0          # decisions in other modules above do reach this slice; below do not
        c = np.zeros(A.shape[1])
        if keep.any():
            c[keep] = np.linalg.lstsq(A[:, keep], b, rcond=None)[0]
        return b - A @ c, c, n


def run_pair(cfg, steps, tol, loss_tol, precision=None, split_after=None, use_graph=False, opt="sgd",
             perturb_affine=0.1, batch=None, check_every=1, lr_schedule=None, noise_mult=None):
    """Step both implementations `steps` times; assert parity at every `check_every`-th step.  Returns the worst
    relative errors seen, for reporting.

    noise_mult (bf16 production kernels): rounding every stored tensor to bf16 makes two evaluations that differ in
    the last bit before a store decorrelate within a few layers (a one-ulp difference of one activation flips the
    rounding of a share of the next layer's outputs), so a path that accumulates in fp32 cannot reproduce the
    oracle's bf16 decisions and its gradients carry an independent draw of the same format noise.  The oracle
    measures that noise itself: e_orc = rel(oracle with bf16 storage, exact oracle) per tensor.  A gradient tensor
    passes if it is within `tol` of the bf16-storage oracle, or if its distance to the exact oracle is at most
    noise_mult * e_orc + tol.  Weights integrate the gradients and are held to the same bar."""
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
    ref = orc.Oracle(layers, split_after, B, cfg["in_shape"], cfg["num_classes"], opt=opt, lr=o["lr"],
                     momentum=o["momentum"], weight_decay=o["weight_decay"], beta1=f32(0.9), beta2=f32(0.999),
                     eps=f32(1e-8), flags=flags)
    gpu = binding.Ddg(layers, split_after, B, cfg["in_shape"], cfg["num_classes"], precision=precision, opt=opt,
                      lr=o["lr"], momentum=o["momentum"], weight_decay=o["weight_decay"], use_graph=use_graph)
    w0 = synth.init_weights(layers, perturb_affine=perturb_affine)
    ref.set_weights(w0.astype(np.float64))
    gpu.set_weights(w0)
    exact = None
    if noise_mult is not None:
        exact = orc.Oracle(layers, split_after, B, cfg["in_shape"], cfg["num_classes"], opt=opt, lr=o["lr"],
                           momentum=o["momentum"], weight_decay=o["weight_decay"], beta1=f32(0.9), beta2=f32(0.999),
                           eps=f32(1e-8), flags=0)
        exact.set_weights(w0.astype(np.float64))
    assert gpu.n_params == ref.n_params and gpu.per_module == ref.per_module
    segs = segments_by_module(layers, split_after)
    worst = dict(loss=0.0, grad=0.0, weight=0.0, tie_steps=0, grad_vs_exact=0.0, oracle_bf16_vs_exact=0.0)
    wbuf = np.empty(gpu.n_params, dtype=np.float32)
    ties = TieExplainer(cfg, B, flags)
    snapshots, batches = {}, {}
    mod_off = np.concatenate([[0], np.cumsum(ref.per_module)]).astype(int)
    for t in range(steps):
        if lr_schedule is not None:
            ref.set_lr(f32(lr_schedule(t))); gpu.set_lr(lr_schedule(t))
        x, y = synth.batch(t, B, cfg["in_shape"], cfg["num_classes"])
        xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
        snapshots[t], batches[t] = ref.get_weights(), (x, y)
        snapshots.pop(t - K - 1, None); batches.pop(t - K - 1, None)
        loss_gpu = gpu.step(xd, yd)
        loss_ref = ref.step(x, y)
        if exact is not None:
            if lr_schedule is not None:
                exact.set_lr(f32(lr_schedule(t)))
            exact.step(x, y)
        if t % check_every and t != steps - 1:
            continue
        dl = abs(loss_gpu - loss_ref) / max(1.0, abs(loss_ref))
        worst["loss"] = max(worst["loss"], dl)
        assert dl <= loss_tol, "step %d: loss %r vs oracle %r" % (t, loss_gpu, loss_ref)
        off = 0
        gpu.get_weights(wbuf)
        wref = ref.get_weights()
        w_ex = exact.get_weights() if exact is not None else None
        for k in range(K):
            gbuf = np.empty(gpu.per_module[k], dtype=np.float32)
            s_gpu = gpu.get_grads(k, gbuf)
            s_ref, g_ref = ref.get_grads(k)
            assert s_gpu == s_ref == (t - K + k + 1 if t - K + k + 1 >= 0 else -1), (t, k, s_gpu, s_ref)
            resid = None
            if exact is not None and s_ref >= 0:
                g_ex = exact.get_grads(k)[1]
                for name, a, b in segs[k]:
                    e_gpu, e_orc = rel(gbuf[a:b], g_ex[a:b]), rel(g_ref[a:b], g_ex[a:b])
                    worst["grad"] = max(worst["grad"], rel(gbuf[a:b], g_ref[a:b]))
                    worst["grad_vs_exact"] = max(worst["grad_vs_exact"], e_gpu)
                    worst["oracle_bf16_vs_exact"] = max(worst["oracle_bf16_vs_exact"], e_orc)
                    assert rel(gbuf[a:b], g_ref[a:b]) <= tol or e_gpu <= noise_mult * e_orc + tol, \
                        "step %d module %d grad %s: %.3e from the exact oracle, format noise %.3e" % (t, k, name, e_gpu, e_orc)
                    e = rel(wbuf[off + a:off + b], wref[off + a:off + b])
                    worst["weight"] = max(worst["weight"], e)
                    # weights integrate the gradients, so they carry the same format noise: same bar
                    ew_gpu = rel(wbuf[off + a:off + b], w_ex[off + a:off + b])
                    ew_orc = rel(wref[off + a:off + b], w_ex[off + a:off + b])
                    assert e <= tol or ew_gpu <= noise_mult * ew_orc + tol, \
                        "step %d module %d weight %s: rel %.3e > %.1e (format noise %.3e)" % (t, k, name, e, tol, ew_orc)
                off += gpu.per_module[k]
                continue
            if s_ref >= 0 and any(rel(gbuf[a:b], g_ref[a:b]) > tol for _, a, b in segs[k]):
                # not within tolerance of the oracle's own ReLU decisions: is it another valid set of decisions?
                resid, coef, n_ties = ties.residual(s_ref, snapshots[s_ref], *batches[s_ref], mod_off[k],
                                                    mod_off[k + 1], gbuf)
                assert n_ties <= ties.max_ties, "too many near-zero ReLU decisions to enumerate (%d)" % n_ties
                assert np.all((np.abs(coef) < 0.05) | (np.abs(coef - 1) < 0.05)), \
                    "step %d module %d: gradient is not a valid set of ReLU decisions %r" % (t, k, coef)
                worst["tie_steps"] += 1
            for name, a, b in segs[k]:
                if s_ref >= 0:
                    if resid is None:
                        e = rel(gbuf[a:b], g_ref[a:b])
                    else:
                        e = float(np.linalg.norm(resid[a:b]) / max(np.linalg.norm(g_ref[a:b]), 1e-12))
                    worst["grad"] = max(worst["grad"], e)
                    assert e <= tol, "step %d module %d grad %s: rel %.3e > %.1e" % (t, k, name, e, tol)
                else:
                    assert not gbuf[a:b].any()
                e = rel(wbuf[off + a:off + b], wref[off + a:off + b])
                worst["weight"] = max(worst["weight"], e)
                assert e <= tol, "step %d module %d weight %s: rel %.3e > %.1e" % (t, k, name, e, tol)
            off += gpu.per_module[k]
    gpu.destroy()
    ref.close()
    if exact is not None:
        exact.close()
    return worst
