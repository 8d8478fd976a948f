"""Plain backpropagation through a layer list with a library autograd (torch, fp64, CPU).

Written independently of the oracle, from the same layer definitions, and used only to pin the oracle:
ordinary BP gradients (Section 2, Eq. 4-5) of the whole network at a given weight vector.
"""
import numpy as np
import torch
import torch.nn.functional as F

from paper_1804_10574_b200 import nets


def forward(layers, w, x, y, bn_eps=1e-5):
    """w: flat torch fp64 tensor (requires_grad), x: [B,C,H,W] fp64, y: int64 labels. Returns mean CE loss."""
    off = 0

    def take(*shape):
        nonlocal off
        n = int(np.prod(shape))
        p = w[off:off + n].reshape(*shape)
        off += n
        return p

    def bn(h, c):
        g, b = take(c), take(c)
        return F.batch_norm(h, None, None, g, b, True, 0.0, bn_eps)

    h = x
    for kind, ci, co, stride, bias, relu in layers:
        if kind == nets.FC:
            h = h.reshape(h.shape[0], -1)
            W = take(co, ci)
            b = take(co) if bias else None
            h = F.linear(h, W, b)
        elif kind == nets.CONV3X3:
            h = F.conv2d(h, take(co, ci, 3, 3), None, stride, 1)
        elif kind == nets.BN:
            h = bn(h, ci)
        elif kind == nets.RELU:
            h = F.relu(h)
        elif kind == nets.GLOBAL_AVGPOOL:
            h = h.mean(dim=(2, 3))
        elif kind in (nets.BASIC_BLOCK, nets.BASIC_BLOCK_PROJ):
            inp = h
            h = F.relu(bn(F.conv2d(inp, take(co, ci, 3, 3), None, stride, 1), co))
            h = bn(F.conv2d(h, take(co, co, 3, 3), None, 1, 1), co)
            if kind == nets.BASIC_BLOCK_PROJ:
                sc = F.conv2d(inp, take(co, ci, 1, 1), None, stride, 0)
            else:
                sc = inp[:, :, ::stride, ::stride]
                if co > ci:
                    sc = F.pad(sc, (0, 0, 0, 0, 0, co - ci))
            h = F.relu(h + sc)
        if relu and kind not in (nets.BASIC_BLOCK, nets.BASIC_BLOCK_PROJ):
            h = F.relu(h)
    assert off == w.numel()
    return F.cross_entropy(h.reshape(h.shape[0], -1), y)


def loss_and_grad(layers, w, x, y):
    wt = torch.tensor(np.asarray(w, dtype=np.float64), requires_grad=True)
    loss = forward(layers, wt, torch.tensor(np.asarray(x, dtype=np.float64)), torch.tensor(np.asarray(y)).long())
    loss.backward()
    return float(loss.detach()), wt.grad.numpy().copy()
