"""Split-position / module-count sweep on one network (Section 5.1: ResNet-8 cut after weighted layer 1, 3, 5 or 7, and
with two to four modules): throughput of the DDG iteration and its loss trajectory per split, on seeded synthetic
CIFAR-shaped batches.  `python -m paper_1804_10574_b200.split_sweep [--net resnet8|resnet56|resnet110] [--steps N]
[--batch B] [--precision bf16|fp32] [--opt adam|sgd] [--projection] [--json]`.  `--projection` runs the same sweep on
the network with 1x1-projection shortcuts on its two shape-changing blocks (the second shortcut type).

A cut may fall only between residual blocks (a shortcut never crosses modules).  The weighted layers of ResNet-8 are
the stem convolution (1), the two convolutions of each of the three blocks (2-3, 4-5, 6-7) and the FC head (8), so
"after layer 1 / 3 / 5 / 7" is after the stem, the first, the second and the third block."""
import argparse
import json

import numpy as np
import torch

from . import binding, nets, synth


def sweep_splits(layers):
    """[(label, split_after)]: every single cut between blocks (after the stem, after each block), then the even
    block splits for K = 3 and K = 4 where the network has enough blocks, and K = 1 (plain backpropagation)."""
    blocks = [i for i, l in enumerate(layers) if l[0] in (nets.BASIC_BLOCK, nets.BASIC_BLOCK_PROJ)]
    out = [("K=1", [])]
    cuts = [blocks[0] - 1] + blocks                       # after the stem's batch norm, after each block
    if len(cuts) > 8:                                      # deep nets: eight evenly spaced single cuts
        cuts = [cuts[int(round(j))] for j in np.linspace(0, len(cuts) - 1, 8)]
    weighted = {nets.FC: 1, nets.CONV3X3: 1, nets.BASIC_BLOCK: 2, nets.BASIC_BLOCK_PROJ: 2}
    for c in cuts:
        n_w = sum(weighted.get(l[0], 0) for l in layers[:c + 1])   # weighted layers (convolutions, FC) before the cut
        out.append(("K=2 after layer %d" % n_w, [c]))
    for K in (3, 4):
        if len(blocks) >= K:
            out.append(("K=%d even" % K, nets.split_even_blocks(layers, K)))
    if len(blocks) == 3:
        out.append(("K=4 stem|b1|b2|b3", [blocks[0] - 1, blocks[0], blocks[1]]))
    return out


def run_one(layers, split_after, batch, in_shape, classes, precision, opt, lr, steps, warmup, n_batches=8):
    d = binding.Ddg(layers, split_after, batch, in_shape, classes, precision=precision, opt=opt, lr=lr, momentum=0.9,
                    weight_decay=5e-4, use_graph=True)
    d.set_weights(synth.init_weights(layers, perturb_affine=0.0))
    data = []
    for t in range(n_batches):
        x, y = synth.batch(t, batch, in_shape, classes)
        data.append((torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()))
    # losses are read (one host sync each) only outside the timed region: the first `warmup` and the last n_batches
    # iterations; the timed iterations queue without a sync, so that consecutive iterations overlap
    first, last = [], []
    for t in range(warmup):
        first.append(d.step(*data[t % n_batches]))
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(warmup, warmup + steps):
        d.step(*data[t % n_batches], want_loss=False)
    d.sync()
    e1.record()
    e1.synchronize()
    for t in range(warmup + steps, warmup + steps + n_batches):
        last.append(d.step(*data[t % n_batches]))
    losses = first + last
    ms = e0.elapsed_time(e1) / steps
    d.destroy()
    return dict(ms_per_step=ms, images_per_s=batch / ms * 1e3, loss_first=float(np.mean(first[:n_batches])),
                loss_last=float(np.mean(last)), finite=bool(np.all(np.isfinite(losses))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--net", default="resnet8", choices=["resnet8", "resnet56", "resnet110"])
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--precision", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--opt", default="adam", choices=["adam", "sgd"])
    ap.add_argument("--lr", type=float, default=None)
    ap.add_argument("--projection", action="store_true", help="1x1-projection shortcuts on the shape-changing blocks")
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    cfg = dict(nets.config(a.net))
    if a.projection:
        units = {"resnet8": 1, "resnet56": 9, "resnet110": 18}[a.net]
        cfg["layers"] = nets.resnet(units, cfg["num_classes"], projection=True)
    lr = a.lr if a.lr is not None else (1e-3 if a.opt == "adam" else 0.01)
    rows = []
    for label, split in sweep_splits(cfg["layers"]):
        r = run_one(cfg["layers"], split, a.batch, cfg["in_shape"], cfg["num_classes"], a.precision, a.opt, lr, a.steps,
                    a.warmup)
        r.update(split=label, split_after=split, K=len(split) + 1)
        rows.append(r)
    if a.json:
        print(json.dumps(dict(net=a.net, batch=a.batch, precision=a.precision, opt=a.opt, lr=lr, steps=a.steps, rows=rows)))
        return
    print("%s%s batch %d %s %s lr %g, %d timed iterations (losses: mean of the first / last 8 iterations, 8 batches cycled)"
          % (a.net, " with projection shortcuts" if a.projection else "", a.batch, a.precision, a.opt, lr, a.steps))
    print("%-22s %2s %10s %12s %10s %10s" % ("split", "K", "ms/iter", "images/s", "loss first", "loss last"))
    for r in rows:
        print("%-22s %2d %10.3f %12.0f %10.4f %10.4f%s" % (r["split"], r["K"], r["ms_per_step"], r["images_per_s"],
                                                          r["loss_first"], r["loss_last"], "" if r["finite"] else "  NOT FINITE"))


if __name__ == "__main__":
    main()
