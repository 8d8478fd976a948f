"""Network specifications and module splits for the DDG workloads (host logic only, no arithmetic).

A network is a list of (kind, c_in, c_out, stride, has_bias, relu_after) tuples.  The architectures are the
CIFAR ResNets of Table 2 of the paper (units 1-1-1 / 9-9-9 / 18-18-18, channels 16-16-32-64, basic blocks
without bottleneck) and a small MLP used as the first parity case.
"""
FC, CONV3X3, BN, RELU, BASIC_BLOCK, GLOBAL_AVGPOOL, BASIC_BLOCK_PROJ = range(7)


def mlp(dims=(64, 128, 128, 128, 10)):
    layers = []
    for i in range(len(dims) - 1):
        last = i == len(dims) - 2
        layers.append((FC, dims[i], dims[i + 1], 1, 1, 0 if last else 1))
    return layers


def resnet(units, num_classes, channels=(16, 16, 32, 64), in_c=3, projection=False):
    """Stem conv3x3+BN+ReLU, three stages of `units` basic blocks, global mean pool, FC head (Table 2).
    projection: the blocks that change the shape (first of stages 2 and 3) take a 1x1-projection shortcut instead of
    the parameter-free one."""
    layers = [(CONV3X3, in_c, channels[0], 1, 0, 0), (BN, channels[0], channels[0], 1, 0, 1)]
    c = channels[0]
    for stage in range(3):
        c_out = channels[stage + 1]
        for u in range(units):
            stride = 2 if (stage > 0 and u == 0) else 1
            proj = projection and (stride != 1 or c != c_out)
            layers.append((BASIC_BLOCK_PROJ if proj else BASIC_BLOCK, c, c_out, stride, 0, 0))
            c = c_out
    layers.append((GLOBAL_AVGPOOL, c, c, 1, 0, 0))
    layers.append((FC, c, num_classes, 1, 1, 0))
    return layers


def split_even_blocks(layers, K):
    """K-1 split indices that cut between residual blocks with (nearly) equal block counts: the first
    (n_blocks mod K) modules get one extra block; the stem stays with module 1, pool+FC with module K."""
    blocks = [i for i, l in enumerate(layers) if l[0] in (BASIC_BLOCK, BASIC_BLOCK_PROJ)]
    n = len(blocks)
    if K < 1 or K > n:
        raise ValueError("cannot cut %d blocks into %d modules" % (n, K))
    base, extra = divmod(n, K)
    splits, used = [], 0
    for k in range(K - 1):
        used += base + (1 if k < extra else 0)
        splits.append(blocks[used - 1])
    return splits


def param_count(layers):
    n = 0
    for kind, ci, co, stride, bias, relu in layers:
        if kind == FC:
            n += ci * co + (co if bias else 0)
        elif kind == CONV3X3:
            n += ci * co * 9
        elif kind == BN:
            n += 2 * ci
        elif kind in (BASIC_BLOCK, BASIC_BLOCK_PROJ):
            n += ci * co * 9 + co * co * 9 + 4 * co + (ci * co if kind == BASIC_BLOCK_PROJ else 0)
    return n


def param_segments(layers):
    """[(layer index, name, offset, shape, fan_in or None)] in the canonical flat order: per layer the conv/FC
    weight ([Cout][Cin][3][3] or [out][in]), bias, BN gamma, BN beta; a block gives conv1.w, bn1.gamma,
    bn1.beta, conv2.w, bn2.gamma, bn2.beta (and proj.w [Cout][Cin] for a projection shortcut)."""
    segs, off = [], 0

    def add(i, name, shape, fan_in):
        nonlocal off
        size = 1
        for s in shape:
            size *= s
        segs.append((i, name, off, tuple(shape), fan_in))
        off += size

    for i, (kind, ci, co, stride, bias, relu) in enumerate(layers):
        if kind == FC:
            add(i, "fc.w", (co, ci), ci)
            if bias:
                add(i, "fc.b", (co,), None)
        elif kind == CONV3X3:
            add(i, "conv.w", (co, ci, 3, 3), 9 * ci)
        elif kind == BN:
            add(i, "bn.gamma", (ci,), None)
            add(i, "bn.beta", (ci,), None)
        elif kind in (BASIC_BLOCK, BASIC_BLOCK_PROJ):
            add(i, "conv1.w", (co, ci, 3, 3), 9 * ci)
            add(i, "bn1.gamma", (co,), None)
            add(i, "bn1.beta", (co,), None)
            add(i, "conv2.w", (co, co, 3, 3), 9 * co)
            add(i, "bn2.gamma", (co,), None)
            add(i, "bn2.beta", (co,), None)
            if kind == BASIC_BLOCK_PROJ:
                add(i, "proj.w", (co, ci), ci)
    return segs


# The five workload configurations (batch, input shape, classes, split, optimiser) used by tests and bench.
def config(name):
    if name == "mlp":
        L = mlp()
        return dict(layers=L, split_after=[1], batch=16, in_shape=(64, 1, 1), num_classes=10, precision="fp32",
                    opt=dict(lr=0.01, momentum=0.0, weight_decay=0.0))
    if name == "resnet8":
        L = resnet(1, 10)
        return dict(layers=L, split_after=[2], batch=32, in_shape=(3, 32, 32), num_classes=10, precision="fp32",
                    opt=dict(lr=0.1, momentum=0.9, weight_decay=5e-4))
    if name == "resnet56":
        L = resnet(9, 10)
        return dict(layers=L, split_after=split_even_blocks(L, 2), batch=128, in_shape=(3, 32, 32),
                    num_classes=10, precision="bf16", opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    if name == "resnet110":
        L = resnet(18, 100)
        return dict(layers=L, split_after=split_even_blocks(L, 4), batch=128, in_shape=(3, 32, 32),
                    num_classes=100, precision="bf16", opt=dict(lr=0.01, momentum=0.9, weight_decay=5e-4))
    raise KeyError(name)
