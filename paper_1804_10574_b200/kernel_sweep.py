"""Per-kernel sweep over the ResNet-110 layer shapes through the single-kernel C-ABI entry points.

    python -m paper_1804_10574_b200.kernel_sweep [--batch 1024] [--only NAME] [--iters 20] [--json] [--warm]

Times every kernel alone with CUDA events on its stream, flushing L2 between launches, and prints the algorithmic
bytes and flops per launch against the measured HBM / bf16 tensor peaks (MEASURED_PEAKS.json at the repository root,
else the fallback 6650 GB/s and 1590 TFLOP/s).  Inputs: bf16 N(0,1) activations and gradients, He-normal filters.
"""
import argparse
import json
import os

import numpy as np
import torch

from . import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def peaks():
    try:
        p = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    except Exception:
        return 6650.0, 1590.0, "fallback"


def timed(fn, iters, flush):
    for _ in range(3):
        fn()
    ts = []
    s = torch.cuda.current_stream()
    for _ in range(iters):
        if flush is not None:
            flush.zero_()
        else:
            torch.cuda._sleep(200000)   # keeps the GPU busy without touching L2 while the host enqueues what follows
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        fn()
        e1.record(s)
        e1.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e-3)
    ts = sorted(ts)
    if len(ts) >= 6:             # event stamps tick every ~2 us: averaging resolves below that, the median cannot
        ts = ts[1:-1]
    return float(np.mean(ts))


def cases(B):
    bf = torch.bfloat16
    out = []

    def conv(H, Ci, Co, st):
        Ho = (H - 1) // st + 1
        x = torch.randn(B, H, H, Ci, device="cuda").to(bf)
        dy = torch.randn(B, Ho, Ho, Co, device="cuda").to(bf)
        w = (torch.randn(Co, Ci, 3, 3, device="cuda") * (2.0 / (9 * Ci)) ** 0.5).to(bf)
        y, dx = torch.empty_like(dy), torch.empty_like(x)
        dw = torch.empty(Co, Ci, 3, 3, device="cuda")
        sc = torch.empty(max(1, binding.conv3x3_wgrad_scratch_elems(B, H, H, Ci, Co, st)), device="cuda")
        flops = 2.0 * 9 * Ci * Co * B * Ho * Ho
        io = (x.numel() + dy.numel()) * 2
        tag = "%d->%d %dx%d s%d" % (Ci, Co, H, H, st)
        tc = binding.tensor_core_path(B, H, H, Ci, Co, st)
        keep = (x, dy, w, y, dx, dw, sc)
        if tc & 1 and st == 1 and Ci == Co:   # as in the training step: filter image arranged beforehand (by the optimiser update)
            pk = torch.empty(binding.conv3x3_packed_bytes(B, H, H, Ci), dtype=torch.uint8, device="cuda")
            binding.conv3x3_pack(w, pk, Ci)
            out.append(("conv_fwd " + tag, lambda: binding.conv3x3_packed(0, x, w, pk, y, B, H, H, Ci), io, flops, 1, keep + (pk,)))
            out.append(("conv_dgrad " + tag, lambda: binding.conv3x3_packed(1, dy, w, pk, dx, B, H, H, Ci), io, flops, 1, keep + (pk,)))
        else:
            out.append(("conv_fwd " + tag, lambda: binding.conv3x3_fwd(1, x, w, y, B, H, H, Ci, Co, st), io, flops, tc & 1, keep))
            out.append(("conv_dgrad " + tag, lambda: binding.conv3x3_dgrad(1, dy, w, dx, B, H, H, Ci, Co, st), io, flops, tc & 1, keep))
        out.append(("conv_wgrad " + tag, lambda: binding.conv3x3_wgrad(1, x, dy, dw, sc, B, H, H, Ci, Co, st), io, flops, (tc >> 1) & 1, keep))

    for H, Ci, Co, st in ((32, 16, 16, 1), (16, 32, 32, 1), (8, 64, 64, 1), (32, 16, 32, 2), (16, 32, 64, 2), (32, 3, 16, 1)):
        conv(H, Ci, Co, st)

    def bn(H, C):
        HW = H * H
        x = torch.randn(B, HW, C, device="cuda").to(bf)
        r, dout = torch.randn_like(x), torch.randn_like(x)
        g, b = torch.ones(C, device="cuda").to(bf), torch.zeros(C, device="cuda").to(bf)
        y, dx = torch.empty_like(x), torch.empty_like(x)
        m, i, dg, db = (torch.empty(C, device="cuda") for _ in range(4))
        sc = torch.zeros(binding.bn_scratch_elems(C), device="cuda")
        keep = (x, r, dout, g, b, y, dx, m, i, dg, db, sc)
        n = x.numel() * 2
        out.append(("bn_relu_residual_fwd C%d %dx%d" % (C, H, H),
                    lambda: binding.bn_fwd(1, x, g, b, r, y, m, i, sc, B, HW, C, 1), 4 * n, 0.0, 0, keep))   # x twice, res, y
        out.append(("bn_relu_bwd C%d %dx%d" % (C, H, H),
                    lambda: binding.bn_bwd(1, dout, y, x, g, m, i, dx, dg, db, sc, B, HW, C, 1), 7 * n, 0.0, 0, keep))

    for H, C in ((32, 16), (16, 32), (8, 64)):
        bn(H, C)

    n = 1733812
    w, v, gr = (torch.randn(n, device="cuda") for _ in range(3))
    wv = torch.empty(n, dtype=bf, device="cuda")
    out.append(("sgd_update 1.73M params", lambda: binding.sgd_update(1, w, v, gr, wv, n, 0.01, 0.9, 5e-4), n * 22, 0.0, 0, (w, v, gr, wv)))
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=1024)
    ap.add_argument("--only", default="")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--json", action="store_true")
    ap.add_argument("--warm", action="store_true", help="do not flush L2 between launches (operands as the previous "
                    "kernel of a training step leaves them)")
    a = ap.parse_args()
    hbm, tf, src = peaks()
    flush = None if a.warm else torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    rows = []
    for name, fn, nbytes, flops, tc, _keep in cases(a.batch):
        if a.only and a.only not in name:
            continue
        dt = timed(fn, a.iters, flush)
        rows.append(dict(kernel=name, tensor_core=bool(tc), us=dt * 1e6, gbs=nbytes / dt / 1e9, hbm_frac=nbytes / dt / 1e9 / hbm,
                         tflops=flops / dt / 1e12, tensor_frac=flops / dt / 1e12 / tf))
    if a.json:
        print(json.dumps(dict(batch=a.batch, peaks=dict(hbm_gbs=hbm, bf16_tflops=tf, source=src), rows=rows)))
        return
    print("batch %d; peaks (%s): HBM %.0f GB/s, bf16 %.0f TFLOP/s" % (a.batch, src, hbm, tf))
    print("%-34s %3s %9s %9s %7s %9s %7s" % ("kernel", "tc", "us", "GB/s", "of HBM", "TFLOP/s", "of bf16"))
    for r in rows:
        print("%-34s %3s %9.1f %9.0f %6.1f%% %9.1f %6.1f%%" % (r["kernel"], "yes" if r["tensor_core"] else "no", r["us"], r["gbs"],
                                                              100 * r["hbm_frac"], r["tflops"], 100 * r["tensor_frac"]))
    if any(r["kernel"].endswith("3->16 32x32 s1") for r in rows):
        print("3->16: the single-kernel entry points take the 3-channel tensor as it is (CUDA-core kernels).  The bf16 training "
              "step never launches these: its input shim stores the image zero-padded to 16 channels and the stem runs on the "
              "16->16 tensor-core kernels above (forward and weight gradient; the input needs no gradient).")


if __name__ == "__main__":
    main()
