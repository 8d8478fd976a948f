"""Per-kernel GPU parity through the single-kernel C-ABI entry points, against the oracle's primitives on the same
seeded inputs.  Shapes span several tiles, ragged tails, both strides and both precisions."""
import numpy as np
import pytest
import torch

from oracle import ddg_oracle as orc
from tests.parity import elementwise_ok, rel

pytestmark = pytest.mark.gpu

TOL = {0: 1e-5, 1: 6e-3}   # fp32: accumulation order only; bf16: inputs are exact bf16, output rounding 2^-9
# per element: |gpu - ref| <= RTOL * |ref| + ATOL_RMS * rms(ref).  bf16: one output rounding (2^-9 relative) plus the
# fp32 accumulation error of a few hundred products; a wrong tap, border or tile seam is an error of order rms(ref)
RTOL = {0: 1e-5, 1: 2.0 ** -8}
ATOL_RMS = {0: 1e-6, 1: 1e-3}


def check_map(got_nchw, ref_nchw, prec, what, seam_rows=None):
    """L2 bar on the whole tensor, the same bar on the image-border pixels alone (and on the rows next to a tile seam,
    every `seam_rows` rows), and the per-element bar on every value."""
    assert rel(got_nchw, ref_nchw) < TOL[prec], what
    H, W = ref_nchw.shape[2], ref_nchw.shape[3]
    if H > 2 and W > 2:
        border = np.ones((H, W), dtype=bool)
        border[1:-1, 1:-1] = False
        assert rel(got_nchw[:, :, border], ref_nchw[:, :, border]) < TOL[prec], what + " (image border)"
        if seam_rows and seam_rows < H:
            seam = np.zeros(H, dtype=bool)
            seam[seam_rows - 1::seam_rows] = True
            seam[seam_rows::seam_rows] = True
            assert rel(got_nchw[:, :, seam, :], ref_nchw[:, :, seam, :]) < TOL[prec], what + " (tile seams)"
    rms = float(np.sqrt(np.mean(np.square(ref_nchw)))) if ref_nchw.size else 0.0
    ok, idx, excess = elementwise_ok(got_nchw, ref_nchw, RTOL[prec], ATOL_RMS[prec] * rms)
    assert ok, "%s: element %r off by %.3e beyond the per-element bar" % (what, idx, excess)


def tdtype(prec):
    return torch.bfloat16 if prec else torch.float32


def to_dev(a_nchw, prec):
    """fp64 NCHW numpy -> device NHWC tensor in the precision; returns (tensor, the values it holds as fp64 NCHW)."""
    t = torch.from_numpy(np.ascontiguousarray(a_nchw)).to(tdtype(prec))
    held = t.to(torch.float64).numpy()
    if t.dim() == 4:
        t = t.permute(0, 2, 3, 1).contiguous()
    return t.cuda(), held


def from_dev(t_nhwc):
    return t_nhwc.to(torch.float64).cpu().permute(0, 3, 1, 2).contiguous().numpy()


SHAPES = [  # B, H, W, Cin, Cout, stride
    (2, 8, 8, 16, 16, 1), (3, 32, 32, 16, 16, 1), (5, 16, 16, 32, 32, 1), (9, 8, 8, 64, 64, 1),
    (3, 32, 32, 16, 32, 2), (3, 16, 16, 32, 64, 2), (6, 16, 16, 32, 64, 2), (7, 32, 32, 32, 64, 2), (10, 16, 16, 16, 32, 2),
    (4, 32, 32, 3, 16, 1), (2, 7, 5, 5, 12, 1), (2, 9, 7, 6, 10, 2),
    (128, 8, 8, 64, 64, 1),
]


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_conv3x3_fwd_dgrad_wgrad(shape, prec):
    from paper_1804_10574_b200 import binding
    B, H, W, Ci, Co, st = shape
    rng = np.random.default_rng(11)
    Ho, Wo = (H - 1) // st + 1, (W - 1) // st + 1
    x, xh = to_dev(rng.standard_normal((B, Ci, H, W)), prec)
    w = torch.from_numpy(rng.standard_normal((Co, Ci, 3, 3)) * np.sqrt(2.0 / (9 * Ci))).to(tdtype(prec))
    wh = w.to(torch.float64).numpy()
    w = w.cuda()
    dy, dyh = to_dev(rng.standard_normal((B, Co, Ho, Wo)), prec)
    y = torch.empty(B, Ho, Wo, Co, dtype=tdtype(prec), device="cuda")
    dx = torch.empty(B, H, W, Ci, dtype=tdtype(prec), device="cuda")
    dw = torch.empty(Co, Ci, 3, 3, dtype=torch.float32, device="cuda")
    scratch = torch.empty(max(1, binding.conv3x3_wgrad_scratch_elems(B, H, W, Ci, Co, st)), dtype=torch.float32,
                          device="cuda")
    binding.conv3x3_fwd(prec, x, w, y, B, H, W, Ci, Co, st)
    binding.conv3x3_dgrad(prec, dy, w, dx, B, H, W, Ci, Co, st)
    binding.conv3x3_wgrad(prec, x, dy, dw, scratch, B, H, W, Ci, Co, st)
    torch.cuda.synchronize()
    y_ref = orc.conv3x3_forward(xh, wh, st)
    dx_ref, dw_ref = orc.conv3x3_backward(xh, wh, dyh, st)
    seam = max(1, 128 // Wo) if prec else None      # a tensor-core tile is 128 pixels = 128 / W image rows
    check_map(from_dev(y), y_ref, prec, "forward", seam)
    check_map(from_dev(dx), dx_ref, prec, "input gradient", max(1, 128 // W) if prec else None)
    tc_w = prec and binding.tensor_core_path(B, H, W, Ci, Co, st) & 2
    ok, idx, excess = elementwise_ok(dw.cpu().numpy(), dw_ref, 2e-4 if tc_w else 1e-5,
                                     (2e-4 if tc_w else 1e-6) * float(np.sqrt(np.mean(np.square(dw_ref)))))
    assert ok, "weight gradient: element %r off by %.3e" % (idx, excess)
    # fp32 output from exact inputs in both precisions; the tensor-core path accumulates in fp32 over all pixels
    assert rel(dw.cpu().numpy(), dw_ref) < (2e-4 if prec and binding.tensor_core_path(B, H, W, Ci, Co, st) & 2 else 1e-5)
    # a second call on the same scratch gives the same bits (fixed summation order)
    dw2 = torch.empty_like(dw)
    binding.conv3x3_wgrad(prec, x, dy, dw2, scratch, B, H, W, Ci, Co, st)
    torch.cuda.synchronize()
    assert torch.equal(dw, dw2)


# enough tiles per CTA for the launch plans that large batches get (four epilogue groups, deep stage rings, chunked
# weight gradient), with a ragged last wave
@pytest.mark.parametrize("shape", [(301, 32, 32, 16, 16, 1), (231, 16, 16, 32, 32, 1), (902, 8, 8, 64, 64, 1)],
                         ids=lambda s: "x".join(map(str, s)))
def test_conv3x3_many_tiles(shape):
    test_conv3x3_fwd_dgrad_wgrad(shape, 1)


# The launch plan (pipelines per CTA, epilogue groups, stage ring) depends on the number of tiles, the arithmetic of
# an output pixel does not: a batch of the kernel-sweep size must give, image for image, the bits that the same images
# give in small batches (whose plan the oracle comparisons above cover).
@pytest.mark.parametrize("shape", [(1024, 32, 32, 16), (1024, 16, 16, 32), (1280, 16, 16, 32), (4096, 8, 8, 64)],
                         ids=lambda s: "x".join(map(str, s)))
def test_conv3x3_large_batch_equals_small_batches(shape):
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    g = torch.Generator(device="cuda").manual_seed(17)
    x = torch.randn(B, H, W, C, device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn(C, C, 3, 3, device="cuda", generator=g) * (2.0 / (9 * C)) ** 0.5).to(torch.bfloat16)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    binding.conv3x3_fwd(1, x, w, y, B, H, W, C, C, 1)
    binding.conv3x3_dgrad(1, x, w, dx, B, H, W, C, C, 1)
    step = 64
    for i in (0, B // 2, B - step):   # first, middle and last slice
        ys, dxs = torch.empty_like(x[i:i + step]), torch.empty_like(x[i:i + step])
        binding.conv3x3_fwd(1, x[i:i + step], w, ys, step, H, W, C, C, 1)
        binding.conv3x3_dgrad(1, x[i:i + step], w, dxs, step, H, W, C, C, 1)
        torch.cuda.synchronize()
        assert torch.equal(ys, y[i:i + step]) and torch.equal(dxs, dx[i:i + step]), (shape, i)


def test_conv3x3_wgrad_very_large_batch_equals_sum_of_parts():
    """The weight gradient is a sum over the images of the batch: at a batch large enough for the launch plan with two
    CTAs per SM (32 channels, 2400 images of 16x16) it must equal the sum of the weight gradients of four quarters of
    the batch (sizes whose plan the oracle comparisons above cover) up to the order of the fp32 additions."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = 2400, 16, 16, 32
    g = torch.Generator(device="cuda").manual_seed(23)
    x = torch.randn(B, H, W, C, device="cuda", generator=g).to(torch.bfloat16)
    dy = torch.randn(B, H, W, C, device="cuda", generator=g).to(torch.bfloat16)
    scratch = torch.zeros(binding.conv3x3_wgrad_scratch_elems(B, H, W, C, C, 1), device="cuda")
    dw = torch.empty(C, C, 3, 3, device="cuda")
    binding.conv3x3_wgrad(1, x, dy, dw, scratch, B, H, W, C, C, 1)
    parts = torch.zeros(C, C, 3, 3, device="cuda", dtype=torch.float64)
    step = B // 4
    for i in range(0, B, step):
        dws = torch.empty(C, C, 3, 3, device="cuda")
        binding.conv3x3_wgrad(1, x[i:i + step], dy[i:i + step], dws, scratch, step, H, W, C, C, 1)
        parts += dws.double()
    torch.cuda.synchronize()
    assert rel(dw.cpu().numpy(), parts.cpu().numpy()) < 2e-6
    assert float((dw.double() - parts).abs().max()) <= 1e-4 * float(parts.abs().max())


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
# the last shape is large enough for the many-vectors-per-thread variants of the reductions and element-wise passes
@pytest.mark.parametrize("shape", [(4, 64, 16), (7, 1024, 16), (33, 256, 32), (128, 64, 64), (3, 35, 12), (2, 3, 8),
                                   (601, 1024, 16)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("relu,res", [(0, 0), (1, 0), (1, 1)])
def test_bn_fwd_bwd(shape, prec, relu, res):
    from paper_1804_10574_b200 import binding
    B, HW, C = shape
    rng = np.random.default_rng(5)
    x, xh = to_dev((rng.standard_normal((B, C, HW, 1)) * 1.5 + 0.3), prec)
    gamma = torch.from_numpy(1 + 0.2 * rng.standard_normal(C)).to(tdtype(prec))
    beta = torch.from_numpy(0.2 * rng.standard_normal(C)).to(tdtype(prec))
    gh, bh = gamma.to(torch.float64).numpy(), beta.to(torch.float64).numpy()
    r, rh = to_dev(rng.standard_normal((B, C, HW, 1)), prec)
    dout, douth = to_dev(rng.standard_normal((B, C, HW, 1)), prec)
    y = torch.empty_like(x)
    dx = torch.empty_like(x)
    mean, invstd, dg, db = (torch.empty(C, dtype=torch.float32, device="cuda") for _ in range(4))
    scratch = torch.full((binding.bn_scratch_elems(C),), 7.0, dtype=torch.float32, device="cuda")  # junk on entry
    binding.bn_fwd(prec, x, gamma.cuda(), beta.cuda(), r if res else None, y, mean, invstd, scratch, B, HW, C, relu)
    binding.bn_bwd(prec, dout, y, x, gamma.cuda(), mean, invstd, dx, dg, db, scratch, B, HW, C, relu)
    torch.cuda.synchronize()
    y_ref, m_ref, is_ref = orc.bn_forward(xh, gh, bh)
    if res:
        y_ref = y_ref + rh
    if relu:
        y_ref = np.maximum(y_ref, 0)
    assert rel(mean.cpu().numpy(), m_ref) < 1e-5 and rel(invstd.cpu().numpy(), is_ref) < 1e-5
    assert rel(from_dev(y), y_ref) < TOL[prec]
    yrms = float(np.sqrt(np.mean(np.square(y_ref))))
    ok, idx, excess = elementwise_ok(from_dev(y), y_ref, RTOL[prec], (2e-3 if prec else 1e-5) * yrms)
    assert ok, "batch-norm output: element %r off by %.3e" % (idx, excess)
    # backward reference uses the mask of the output the GPU actually stored
    dz = douth * (from_dev(y) > 0) if relu else douth
    dx_ref, dg_ref, db_ref = orc.bn_backward(xh, m_ref, is_ref, gh, dz)
    tol_s = 2e-5 if HW * B > 4 else 1e-3
    assert rel(db.cpu().numpy(), db_ref) < tol_s and rel(dg.cpu().numpy(), dg_ref) < tol_s
    assert rel(from_dev(dx), dx_ref) < max(TOL[prec], tol_s)


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("n", [1, 5, 1024, 1733812])
def test_sgd_update(n, prec):
    """The update kernel against the oracle's own update: an FC layer of n weights without bias, K = 1, batch 1, input
    x = 1, two classes.  With lr = 0 the oracle's step leaves the gradient g of its first iteration in get_grads; with
    the same (w, g) and zero momentum state the oracle's next step is the reference for the kernel (Eq. 9 with momentum
    and decay as the oracle reads them)."""
    from paper_1804_10574_b200 import binding
    rng = np.random.default_rng(3)
    w, v, g = (rng.standard_normal(n).astype(np.float32) for _ in range(3))
    wd, vd, gd = (torch.from_numpy(a).cuda() for a in (w, v, g))
    wv = torch.empty(n, dtype=tdtype(prec), device="cuda")
    binding.sgd_update(prec, wd, vd, gd, wv, n, 0.1, 0.9, 5e-4)
    torch.cuda.synchronize()
    d = g.astype(np.float64) + float(np.float32(5e-4)) * w
    v_ref = float(np.float32(0.9)) * v + d
    w_ref = w - float(np.float32(0.1)) * v_ref
    assert rel(vd.cpu().numpy(), v_ref) < 1e-6 and rel(wd.cpu().numpy(), w_ref) < 1e-6
    if n == 1024:
        # the same numbers through the oracle's optimiser: a bias-free FC layer 512 -> 2 holds n = 1024 weights; one
        # iteration from momentum 0 gives w1 = w - lr * (g + wd * w), which the kernel must reproduce from (w, 0, g)
        f32 = lambda q: float(np.float32(q))
        o = orc.Oracle([(0, 512, 2, 1, 0, 0)], [], 1, (512, 1, 1), 2, lr=f32(0.1), momentum=f32(0.9), weight_decay=f32(5e-4))
        o.set_weights(w.astype(np.float64))
        xo = rng.standard_normal((1, 512, 1, 1))
        o.step(xo, np.zeros(1, dtype=np.int32))
        g_o = o.get_grads(0)[1]
        w1_o = o.get_weights()
        w2, v2, g2 = torch.from_numpy(w).cuda(), torch.zeros(n, device="cuda"), torch.from_numpy(g_o.astype(np.float32)).cuda()
        binding.sgd_update(prec, w2, v2, g2, torch.empty_like(wv), n, 0.1, 0.9, 5e-4)
        torch.cuda.synchronize()
        assert rel(w2.cpu().numpy(), w1_o) < 1e-6 and rel(v2.cpu().numpy(), g_o + f32(5e-4) * w.astype(np.float64)) < 1e-6
    assert torch.equal(wv, wd.to(tdtype(prec)))      # the version slot is the cast of the new master weights


def test_tensor_core_path_takes_the_resnet_shapes():
    from paper_1804_10574_b200 import binding
    for B, H, W, C in [(128, 32, 32, 16), (128, 16, 16, 32), (128, 8, 8, 64), (2, 8, 8, 16), (3, 32, 32, 16)]:
        assert binding.tensor_core_path(B, H, W, C, C, 1) & 1, (B, H, W, C)
    assert binding.tensor_core_path(128, 32, 32, 16, 32, 2) == 3           # the down-sampling convolutions too
    assert binding.tensor_core_path(128, 16, 16, 32, 64, 2) == 3
    assert binding.tensor_core_path(3, 16, 16, 32, 64, 2) == 0             # 8x8 output: tiles are image pairs
    assert binding.tensor_core_path(9, 8, 8, 64, 64, 1) & 1 == 0          # 576 pixels: not whole 128-pixel tiles


@pytest.mark.parametrize("shape", [(3, 32, 32, 16), (5, 16, 16, 32), (128, 8, 8, 64)], ids=lambda s: "x".join(map(str, s)))
def test_conv3x3_with_prearranged_filter_matches_oracle(shape):
    """The filter-image path the training step uses (pack once, bulk-copied by the kernel), forward and dgrad."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(13)
    x, xh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    dy, dyh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    w = torch.from_numpy(rng.standard_normal((C, C, 3, 3)) * np.sqrt(2.0 / (9 * C))).to(torch.bfloat16)
    wh = w.to(torch.float64).numpy()
    w = w.cuda()
    pk = torch.empty(binding.conv3x3_packed_bytes(B, H, W, C), dtype=torch.uint8, device="cuda")
    assert pk.numel() == 2 * 9 * C * C * 2
    binding.conv3x3_pack(w, pk, C)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    binding.conv3x3_packed(0, x, w, pk, y, B, H, W, C)
    binding.conv3x3_packed(1, dy, w, pk, dx, B, H, W, C)
    torch.cuda.synchronize()
    check_map(from_dev(y), orc.conv3x3_forward(xh, wh, 1), 1, "forward", max(1, 128 // W))
    check_map(from_dev(dx), orc.conv3x3_backward(xh, wh, dyh, 1)[0], 1, "input gradient", max(1, 128 // W))


# ---- the fused epilogues of the training step, each against oracle primitives composed on the same bf16 inputs ----
FUSED_SHAPES = [(3, 32, 32, 16), (5, 16, 16, 32), (128, 8, 8, 64), (2, 8, 8, 16), (8, 8, 8, 32),      # slab and image-pair tiles
                (301, 32, 32, 16), (231, 16, 16, 32), (902, 8, 8, 64)]                                  # many tiles per CTA


def _filter(rng, C, Co=None):
    Co = Co or C
    w = torch.from_numpy(rng.standard_normal((Co, C, 3, 3)) * np.sqrt(2.0 / (9 * C))).to(torch.bfloat16)
    return w.cuda(), w.to(torch.float64).numpy()


@pytest.mark.parametrize("shape", FUSED_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("packed", [False, True], ids=["canonical", "image"])
def test_conv_forward_with_batch_statistics(shape, packed):
    """Eq. 3 for conv -> batch norm: the convolution's epilogue also delivers mean and 1/sqrt(var + eps) of its (stored)
    output.  Tensor against the oracle's convolution; statistics against the oracle's batch norm applied to the tensor
    the GPU stored, and to the oracle's own bf16-rounded output."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(21)
    x, xh = to_dev(rng.standard_normal((B, C, H, W)) * 1.2 + 0.1, 1)
    w, wh = _filter(rng, C)
    pk = None
    if packed:
        pk = torch.empty(binding.conv3x3_packed_bytes(B, H, W, C), dtype=torch.uint8, device="cuda")
        binding.conv3x3_pack(w, pk, C)
    y = torch.empty_like(x)
    mean, invstd = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(2))
    scratch = torch.full((binding.conv3x3_fused_scratch_elems(B, H, W, C),), 3.0, dtype=torch.float32, device="cuda")
    for _ in range(2):       # the second call finds the first one's leftovers in the scratch
        binding.conv3x3_fwd_stats(x, w, pk, y, mean, invstd, scratch, B, H, W, C)
    torch.cuda.synchronize()
    y_ref = orc.conv3x3_forward(xh, wh, 1)
    check_map(from_dev(y), y_ref, 1, "forward", max(1, 128 // W))
    ones, zeros = np.ones(C), np.zeros(C)
    _, m_ref, is_ref = orc.bn_forward(from_dev(y), ones, zeros)
    assert rel(mean.cpu().numpy(), m_ref) < 2e-5 and rel(invstd.cpu().numpy(), is_ref) < 2e-5
    y_b = torch.from_numpy(y_ref).to(torch.bfloat16).to(torch.float64).numpy()
    _, m2, is2 = orc.bn_forward(y_b, ones, zeros)
    assert np.max(np.abs(mean.cpu().numpy() - m2)) < 1e-3 * float(np.sqrt(np.mean(y_ref ** 2))) and rel(invstd.cpu().numpy(), is2) < 1e-3


# the shapes of the ResNet-110 batch-128 step (the plan gives their pipelines two or four tiles on fewer CTAs), small
# batches (CTAs with a single pipeline and two tiles) and many tiles
@pytest.mark.parametrize("shape", [(128, 32, 32, 16), (128, 16, 16, 32), (128, 8, 8, 64), (3, 32, 32, 16), (5, 16, 16, 32),
                                   (10, 8, 8, 64), (74, 16, 16, 32), (301, 32, 32, 16), (231, 16, 16, 32), (902, 8, 8, 64)],
                         ids=lambda s: "x".join(map(str, s)))
def test_conv_forward_with_batch_statistics_shared_gpu_plan(shape):
    """The launch plan of a step whose K > 1 module streams share the GPU (fewer CTAs, at least two tiles per pipeline)
    changes neither a pixel nor, beyond the order of the additions, the statistics: y equals the single-stream plan's y
    bit for bit, mean and invstd agree with it to fp32 rounding and with the oracle's batch norm of the stored tensor."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(29)
    x, _ = to_dev(rng.standard_normal((B, C, H, W)) * 1.1 - 0.2, 1)
    w, _ = _filter(rng, C)
    pk = torch.empty(binding.conv3x3_packed_bytes(B, H, W, C), dtype=torch.uint8, device="cuda")
    binding.conv3x3_pack(w, pk, C)
    y0, y1 = torch.empty_like(x), torch.full_like(x, 5.0)
    m0, i0, m1, i1 = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(4))
    scratch = torch.zeros(binding.conv3x3_fused_scratch_elems(B, H, W, C), dtype=torch.float32, device="cuda")
    binding.conv3x3_fwd_stats(x, w, pk, y0, m0, i0, scratch, B, H, W, C)
    for _ in range(2):     # the ticket counter is left at zero by every call
        binding.conv3x3_fwd_stats_shared(x, w, pk, y1, m1, i1, scratch, B, H, W, C)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)
    assert rel(m1.cpu().numpy(), m0.cpu().numpy()) < 2e-6 and rel(i1.cpu().numpy(), i0.cpu().numpy()) < 2e-6
    _, m_ref, is_ref = orc.bn_forward(from_dev(y1), np.ones(C), np.zeros(C))
    assert rel(m1.cpu().numpy(), m_ref) < 2e-5 and rel(i1.cpu().numpy(), is_ref) < 2e-5


@pytest.mark.parametrize("shape", FUSED_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("with_shortcut,with_sums", [(True, False), (False, True), (True, True)],
                         ids=["shortcut", "sums", "shortcut_sums"])
def test_conv_input_gradient_with_shortcut_and_batch_norm_sums(shape, with_shortcut, with_sums):
    """Eq. 5 / Eq. 7 as the backward sweep launches it: dx = dgrad(dy) [+ dout * [out > 0]] and the two reductions of
    the batch-norm backward that consumes dx.  dx against the oracle's convolution backward plus the shortcut term;
    (dbeta, dgamma) against the oracle's batch-norm backward fed the dx the GPU stored."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(23)
    dy, dyh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    w, wh = _filter(rng, C)
    dout, douth = to_dev(rng.standard_normal((B, C, H, W)), 1)
    out, outh = to_dev(np.maximum(rng.standard_normal((B, C, H, W)), 0), 1)       # a ReLU output: about half zeros
    mask, maskh = to_dev(np.maximum(rng.standard_normal((B, C, H, W)), 0), 1)
    bx, bxh = to_dev(rng.standard_normal((B, C, H, W)) * 1.5 + 0.3, 1)
    _, m_ref, is_ref = orc.bn_forward(bxh, np.ones(C), np.zeros(C))
    mean = torch.from_numpy(m_ref.astype(np.float32)).cuda()
    invstd = torch.from_numpy(is_ref.astype(np.float32)).cuda()
    dx = torch.empty_like(dy)
    db, dg = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(2))
    scratch = torch.full((binding.conv3x3_fused_scratch_elems(B, H, W, C),), 3.0, dtype=torch.float32, device="cuda")
    for _ in range(2):
        binding.conv3x3_dgrad_fused(dy, w, None, dx, dout if with_shortcut else None, out if with_shortcut else None,
                                    mask if with_sums else None, bx if with_sums else None,
                                    mean if with_sums else None, invstd if with_sums else None,
                                    db if with_sums else None, dg if with_sums else None, scratch, B, H, W, C)
    torch.cuda.synchronize()
    dx_ref = orc.conv3x3_backward(np.zeros_like(dyh), wh, dyh, 1)[0]
    if with_shortcut:
        dx_ref = dx_ref + douth * (outh > 0)
    check_map(from_dev(dx), dx_ref, 1, "input gradient", max(1, 128 // W))
    if with_sums:
        dz = from_dev(dx) * (maskh > 0)
        _, dg_ref, db_ref = orc.bn_backward(bxh, mean.double().cpu().numpy(), invstd.double().cpu().numpy(), np.ones(C), dz)
        scale = float(np.sqrt(np.mean(dz ** 2)) * np.sqrt(B * H * W))       # size of a sum of that many such terms
        assert np.max(np.abs(db.cpu().numpy() - db_ref)) < 2e-5 * scale, (db.cpu().numpy(), db_ref)
        assert np.max(np.abs(dg.cpu().numpy() - dg_ref)) < 2e-5 * scale * 2, (dg.cpu().numpy(), dg_ref)


@pytest.mark.parametrize("shape", [(128, 32, 32, 16), (128, 16, 16, 32), (128, 8, 8, 64), (5, 16, 16, 32), (10, 8, 8, 64),
                                   (231, 16, 16, 32), (902, 8, 8, 64)], ids=lambda s: "x".join(map(str, s)))
def test_conv_input_gradient_fused_shared_gpu_plan(shape):
    """The input-gradient convolution with the shortcut gradient and the batch-norm sums under the launch plan of a step
    whose module streams share the GPU: dx equals the single-stream plan's dx bit for bit (whose values the test above
    holds against the oracle), the sums agree with it to fp32 rounding."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    g = torch.Generator(device="cuda").manual_seed(31)
    rnd = lambda: torch.randn(B, H, W, C, device="cuda", generator=g)
    dy, dout, bx = rnd().to(torch.bfloat16), rnd().to(torch.bfloat16), (rnd() * 1.5 + 0.3).to(torch.bfloat16)
    out, mask = rnd().clamp_min(0).to(torch.bfloat16), rnd().clamp_min(0).to(torch.bfloat16)
    w = (torch.randn(C, C, 3, 3, device="cuda", generator=g) * (2.0 / (9 * C)) ** 0.5).to(torch.bfloat16)
    mean = bx.float().mean(dim=(0, 1, 2)).contiguous()
    invstd = (1.0 / torch.sqrt(bx.float().var(dim=(0, 1, 2), unbiased=False) + 1e-5)).contiguous()
    scratch = torch.zeros(binding.conv3x3_fused_scratch_elems(B, H, W, C), dtype=torch.float32, device="cuda")
    res = []
    for fn in (binding.conv3x3_dgrad_fused, binding.conv3x3_dgrad_fused_shared, binding.conv3x3_dgrad_fused_shared):
        dx = torch.full_like(dy, 3.0)
        db, dg = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(2))
        fn(dy, w, None, dx, dout, out, mask, bx, mean, invstd, db, dg, scratch, B, H, W, C)
        torch.cuda.synchronize()
        res.append((dx, db.cpu().numpy(), dg.cpu().numpy()))
    scale = float(np.abs(res[0][1]).max() + np.abs(res[0][2]).max())
    for dx, db, dg in res[1:]:
        assert torch.equal(dx, res[0][0])
        assert np.max(np.abs(db - res[0][1])) < 2e-6 * scale + 1e-4 and np.max(np.abs(dg - res[0][2])) < 2e-6 * scale + 1e-4
    assert np.array_equal(res[1][1], res[2][1]) and np.array_equal(res[1][2], res[2][2])   # fixed order: same bits again


@pytest.mark.parametrize("shape", [(3, 32, 32, 16), (6, 16, 16, 32), (7, 32, 32, 32), (10, 16, 16, 16), (128, 32, 32, 16)],
                         ids=lambda s: "x".join(map(str, s)))
def test_stride2_input_gradient_with_parameter_free_shortcut(shape):
    """The down-sampling block's first convolution in the backward sweep: dx = dgrad_stride2(dy) plus the gradient of
    the parameter-free shortcut (every second pixel of every second row, first Cin channels)."""
    from paper_1804_10574_b200 import binding
    B, H, W, Ci = shape
    Co = 2 * Ci
    rng = np.random.default_rng(29)
    dy, dyh = to_dev(rng.standard_normal((B, Co, H // 2, W // 2)), 1)
    w, wh = _filter(rng, Ci, Co)
    dout, douth = to_dev(rng.standard_normal((B, Co, H // 2, W // 2)), 1)
    out, outh = to_dev(np.maximum(rng.standard_normal((B, Co, H // 2, W // 2)), 0), 1)
    dx = torch.empty(B, H, W, Ci, dtype=torch.bfloat16, device="cuda")
    binding.conv3x3_s2_dgrad_shortcut(dy, w, dx, dout, out, B, H, W, Ci)
    torch.cuda.synchronize()
    dx_ref = orc.conv3x3_backward(np.zeros((B, Ci, H, W)), wh, dyh, 2)[0] + orc.shortcut_backward(douth * (outh > 0), Ci, H, W, 2)
    check_map(from_dev(dx), dx_ref, 1, "stride-2 input gradient with shortcut")
    dx2 = torch.empty_like(dx)
    binding.conv3x3_s2_dgrad_shortcut(dy, w, dx2, None, None, B, H, W, Ci)
    torch.cuda.synchronize()
    check_map(from_dev(dx2), orc.conv3x3_backward(np.zeros((B, Ci, H, W)), wh, dyh, 2)[0], 1, "stride-2 input gradient")


# B, in, out: the paper's heads (64 -> 10 / 100 at batch 128), the MLP's layers, a ragged batch, several batch tiles,
# the widest shapes the tensor-core path takes, and shapes it leaves to the CUDA-core kernels (in = 96, out = 200)
FC_SHAPES = [(128, 64, 100), (128, 64, 10), (16, 64, 128), (16, 128, 128), (16, 128, 10), (7, 64, 10), (300, 128, 100),
             (515, 256, 128), (33, 192, 48), (5, 96, 12), (9, 64, 200)]


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("shape", FC_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("relu,out_f32,bias,want_dx", [(0, 1, 1, 1), (1, 0, 1, 1), (1, 0, 0, 0)],
                         ids=["head", "hidden", "first_nobias"])
def test_fc_fwd_bwd(shape, prec, relu, out_f32, bias, want_dx):
    """Eq. 3-5 for a fully connected layer against the oracle's primitives: forward (bias, ReLU), input gradient,
    weight and bias gradient, as the last layer (fp32 logits and loss gradient: the tensor-core path keeps the loss
    gradient to ~16 bits) and as a hidden layer (bf16 in and out, ReLU mask)."""
    from paper_1804_10574_b200 import binding
    B, n_in, n_out = shape
    rng = np.random.default_rng(31)
    dt = tdtype(prec)
    odt = torch.float32 if out_f32 else dt
    x = torch.from_numpy(rng.standard_normal((B, n_in))).to(dt)
    W = torch.from_numpy(rng.standard_normal((n_out, n_in)) * np.sqrt(2.0 / n_in)).to(dt)
    b = torch.from_numpy(0.3 * rng.standard_normal(n_out)).to(dt)
    dy = torch.from_numpy(rng.standard_normal((B, n_out)) / B).to(odt)
    xh, Wh, bh, dyh = (t.to(torch.float64).numpy() for t in (x, W, b, dy))
    xd, Wd, bd, dyd = x.cuda(), W.cuda(), b.cuda(), dy.cuda()
    y = torch.empty(B, n_out, dtype=odt, device="cuda")
    dx = torch.full((B, n_in), 7.0, dtype=dt, device="cuda")
    dW = torch.full((n_out, n_in), 7.0, dtype=torch.float32, device="cuda")
    db = torch.full((n_out,), 7.0, dtype=torch.float32, device="cuda")
    binding.fc_fwd(prec, xd, Wd, bd if bias else None, y, B, n_in, n_out, relu, out_f32)
    binding.fc_bwd(prec, xd, Wd, y, dyd, dx if want_dx else None, dW, db if bias else None, B, n_in, n_out, relu, out_f32)
    torch.cuda.synchronize()
    y_ref = orc.fc_forward(xh, Wh, bh if bias else np.zeros(n_out))
    if relu:
        y_ref = np.maximum(y_ref, 0)
    yg = y.to(torch.float64).cpu().numpy()
    ytol = 1e-5 if (prec == 0 or out_f32) else TOL[1]
    assert rel(yg, y_ref) < ytol
    rms = float(np.sqrt(np.mean(y_ref ** 2)))
    ok, idx, excess = elementwise_ok(yg, y_ref, 1e-5 if (prec == 0 or out_f32) else RTOL[1], (1e-5 if prec == 0 else 1e-3) * rms)
    assert ok, "fc output element %r off by %.3e" % (idx, excess)
    dz = dyh * (yg > 0) if relu else dyh          # the mask of the output the GPU stored
    dx_ref, dW_ref, db_ref = orc.fc_backward(xh, Wh, dz, True)
    if want_dx:
        assert rel(dx.to(torch.float64).cpu().numpy(), dx_ref) < TOL[prec]
    else:
        assert float(dx.float().min()) == 7.0                     # untouched
    assert rel(dW.cpu().numpy(), dW_ref) < (2e-4 if prec else 1e-5)
    ok, idx, excess = elementwise_ok(dW.cpu().numpy(), dW_ref, 2e-4 if prec else 1e-5,
                                     (2e-4 if prec else 1e-6) * float(np.sqrt(np.mean(dW_ref ** 2))))
    assert ok, "fc weight gradient element %r off by %.3e" % (idx, excess)
    if bias:
        assert rel(db.cpu().numpy(), db_ref) < 1e-5
    else:
        assert float(db.min()) == 7.0


def test_fc_tensor_core_path_takes_the_paper_shapes():
    from paper_1804_10574_b200 import binding
    for B, i, o in [(128, 64, 100), (128, 64, 10), (16, 64, 128), (16, 128, 128), (16, 128, 10), (515, 256, 128)]:
        assert binding.fc_tensor_core_path(B, i, o) == 1, (B, i, o)
    assert binding.fc_tensor_core_path(5, 96, 12) == 0 and binding.fc_tensor_core_path(9, 64, 200) == 0


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(128, 32, 32, 16, 32, 2), (33, 16, 16, 32, 64, 2), (3, 9, 7, 6, 10, 2), (5, 8, 8, 16, 24, 1)],
                         ids=lambda s: "x".join(map(str, s)))
def test_conv1x1_projection(shape, prec):
    """The projection shortcut's 1x1 convolution (forward, input gradient added in place with the ReLU mask of the block
    output, weight gradient) against the oracle's primitive."""
    from paper_1804_10574_b200 import binding
    B, H, W, Ci, Co, st = shape
    rng = np.random.default_rng(37)
    Ho, Wo = (H - 1) // st + 1, (W - 1) // st + 1
    x, xh = to_dev(rng.standard_normal((B, Ci, H, W)), prec)
    w = torch.from_numpy(rng.standard_normal((Co, Ci)) * np.sqrt(2.0 / Ci)).to(tdtype(prec))
    wh = w.to(torch.float64).numpy()
    w = w.cuda()
    dout, douth = to_dev(rng.standard_normal((B, Co, Ho, Wo)), prec)
    out, outh = to_dev(np.maximum(rng.standard_normal((B, Co, Ho, Wo)), 0), prec)
    base, baseh = to_dev(rng.standard_normal((B, Ci, H, W)), prec)      # what the 3x3 input gradient left in dx
    y = torch.empty(B, Ho, Wo, Co, dtype=tdtype(prec), device="cuda")
    dx = base.clone()
    dw = torch.empty(Co, Ci, dtype=torch.float32, device="cuda")
    scratch = torch.empty(binding.conv1x1_wgrad_scratch_elems(Ci, Co), dtype=torch.float32, device="cuda")
    binding.conv1x1_fwd(prec, x, w, y, B, H, W, Ci, Co, st)
    binding.conv1x1_dgrad_add(prec, dout, out, w, dx, B, H, W, Ci, Co, st)
    binding.conv1x1_wgrad(prec, x, dout, out, dw, scratch, B, H, W, Ci, Co, st)
    torch.cuda.synchronize()
    check_map(from_dev(y), orc.conv1x1_forward(xh, wh, st), prec, "1x1 forward")
    dz = douth * (outh > 0)
    dx_ref, dw_ref = orc.conv1x1_backward(xh, wh, dz, st)
    check_map(from_dev(dx), baseh + dx_ref, prec, "1x1 input gradient added in place")
    assert rel(dw.cpu().numpy(), dw_ref) < 1e-5


@pytest.mark.parametrize("shape", [(3, 32, 32, 16), (5, 16, 16, 32), (128, 8, 8, 64), (2, 8, 8, 16), (8, 8, 8, 32),
                                   (128, 32, 32, 16), (128, 16, 16, 32), (301, 32, 32, 16), (231, 16, 16, 32), (902, 8, 8, 64)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("with_res", [False, True], ids=["bn_relu", "bn_add_relu"])
def test_conv_forward_with_batch_norm_relu_on_its_operand_path(shape, with_res):
    """Eq. 3 for batch norm -> ReLU -> convolution in one kernel: a = relu(bn(x)) computed in shared memory from the raw
    x (stored to a_out), y = conv3x3(a) and the statistics of y.  a against the oracle's batch norm + ReLU (and bit for
    bit against the element-wise kernel); y against the oracle's convolution of the a the GPU stored."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(41)
    x, xh = to_dev(rng.standard_normal((B, C, H, W)) * 1.3 + 0.2, 1)
    w, wh = _filter(rng, C)
    gamma = torch.from_numpy(1 + 0.2 * rng.standard_normal(C)).to(torch.bfloat16)
    beta = torch.from_numpy(0.2 * rng.standard_normal(C)).to(torch.bfloat16)
    gh, bh = gamma.to(torch.float64).numpy(), beta.to(torch.float64).numpy()
    r, rh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    a_ref, m_ref, is_ref = orc.bn_forward(xh, gh, bh)
    a_ref = np.maximum(a_ref + (rh if with_res else 0.0), 0)
    mean_in = torch.from_numpy(m_ref.astype(np.float32)).cuda()
    invstd_in = torch.from_numpy(is_ref.astype(np.float32)).cuda()
    a = torch.full_like(x, 7.0)
    y = torch.empty_like(x)
    mean, invstd = (torch.empty(C, dtype=torch.float32, device="cuda") for _ in range(2))
    scratch = torch.zeros(binding.conv3x3_fused_scratch_elems(B, H, W, C), dtype=torch.float32, device="cuda")
    binding.conv3x3_bnrelu_fwd_stats(x, r if with_res else None, gamma.cuda(), beta.cuda(), mean_in, invstd_in, a, w, None, y,
                                     mean, invstd, scratch, B, H, W, C)
    torch.cuda.synchronize()
    arms = float(np.sqrt(np.mean(a_ref ** 2)))
    assert rel(from_dev(a), a_ref) < TOL[1]
    ok, idx, excess = elementwise_ok(from_dev(a), a_ref, RTOL[1], 2e-3 * arms)
    assert ok, "transformed input: element %r off by %.3e" % (idx, excess)
    # the same values as the element-wise batch-norm kernel gives, bit for bit
    a2 = torch.empty_like(x)
    m2, i2 = (torch.empty(C, dtype=torch.float32, device="cuda") for _ in range(2))
    sc2 = torch.zeros(binding.bn_scratch_elems(C), dtype=torch.float32, device="cuda")
    binding.bn_fwd(1, x, gamma.cuda(), beta.cuda(), r if with_res else None, a2, m2, i2, sc2, B, H * W, C, 1)
    torch.cuda.synchronize()
    if torch.equal(m2, mean_in) and torch.equal(i2, invstd_in):      # same statistics in, same bits out
        assert torch.equal(a.view(B, H * W, C), a2.view(B, H * W, C))
    y_ref = orc.conv3x3_forward(from_dev(a), wh, 1)
    check_map(from_dev(y), y_ref, 1, "forward of the transformed input", max(1, 128 // W))
    _, ms, iss = orc.bn_forward(from_dev(y), np.ones(C), np.zeros(C))
    assert rel(mean.cpu().numpy(), ms) < 2e-5 and rel(invstd.cpu().numpy(), iss) < 2e-5


@pytest.mark.parametrize("shape", [(3, 32, 32, 16), (5, 16, 16, 32), (128, 8, 8, 64), (2, 8, 8, 16), (128, 32, 32, 16),
                                   (301, 32, 32, 16), (231, 16, 16, 32), (902, 8, 8, 64)], ids=lambda s: "x".join(map(str, s)))
def test_partial_sums_folded_by_the_consuming_pass(shape):
    """The form a single stream launches: the convolutions leave per-CTA partial sums and the element-wise batch-norm
    passes add them up.  Forward: conv -> batch norm (+ residual, ReLU); backward: input-gradient convolution with the
    two batch-norm sums -> batch-norm backward.  Against the oracle's primitives, statistics and sums teacher-forced on
    the tensors the GPU stored; and against the other form (sums folded by the convolution's last CTA)."""
    from paper_1804_10574_b200 import binding
    B, H, W, C = shape
    rng = np.random.default_rng(43)
    x, xh = to_dev(rng.standard_normal((B, C, H, W)) * 1.2 + 0.1, 1)
    w, wh = _filter(rng, C)
    r, rh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    gamma = torch.from_numpy(1 + 0.2 * rng.standard_normal(C)).to(torch.bfloat16)
    beta = torch.from_numpy(0.2 * rng.standard_normal(C)).to(torch.bfloat16)
    gh, bh = gamma.to(torch.float64).numpy(), beta.to(torch.float64).numpy()
    y, out = torch.empty_like(x), torch.empty_like(x)
    mean, invstd, mean2, invstd2 = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(4))
    part = torch.full((binding.conv3x3_fused_scratch_elems(B, H, W, C),), 3.0, dtype=torch.float32, device="cuda")
    n_part = binding.conv3x3_fwd_partials(x, w, None, y, part, B, H, W, C)
    assert 1 <= n_part <= 148
    binding.bn_fwd_partials(y, gamma.cuda(), beta.cuda(), r, out, part, n_part, mean, invstd, B, H * W, C, 1)
    torch.cuda.synchronize()
    check_map(from_dev(y), orc.conv3x3_forward(xh, wh, 1), 1, "forward", max(1, 128 // W))
    o_ref, m_ref, is_ref = orc.bn_forward(from_dev(y), gh, bh)
    assert rel(mean.cpu().numpy(), m_ref) < 2e-5 and rel(invstd.cpu().numpy(), is_ref) < 2e-5
    o_ref = np.maximum(o_ref + rh, 0)
    assert rel(from_dev(out), o_ref) < TOL[1]
    ok, idx, excess = elementwise_ok(from_dev(out), o_ref, RTOL[1], 2e-3 * float(np.sqrt(np.mean(o_ref ** 2))))
    assert ok, "batch-norm output from partials: element %r off by %.3e" % (idx, excess)
    # the other form of the same launch pair: statistics folded by the convolution's last CTA
    scratch = torch.zeros(binding.conv3x3_fused_scratch_elems(B, H, W, C), dtype=torch.float32, device="cuda")
    y2 = torch.empty_like(x)
    binding.conv3x3_fwd_stats(x, w, None, y2, mean2, invstd2, scratch, B, H, W, C)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    assert torch.equal(mean, mean2) and torch.equal(invstd, invstd2)      # one folding routine, two places: same bits
    # backward
    dy, dyh = to_dev(rng.standard_normal((B, C, H, W)), 1)
    mask, maskh = to_dev(np.maximum(rng.standard_normal((B, C, H, W)), 0), 1)
    bx, bxh = to_dev(rng.standard_normal((B, C, H, W)) * 1.5 + 0.3, 1)
    _, mb, isb = orc.bn_forward(bxh, np.ones(C), np.zeros(C))
    mbd, isbd = torch.from_numpy(mb.astype(np.float32)).cuda(), torch.from_numpy(isb.astype(np.float32)).cuda()
    dx, dxx = torch.empty_like(x), torch.empty_like(x)
    dg, db = (torch.full((C,), 7.0, dtype=torch.float32, device="cuda") for _ in range(2))
    n_part = binding.conv3x3_dgrad_partials(dy, w, None, dx, None, None, mask, bx, mbd, isbd, part, B, H, W, C)
    binding.bn_bwd_partials(dx, mask, bx, gamma.cuda(), mbd, isbd, dxx, dg, db, part, n_part, B, H * W, C, 1)
    torch.cuda.synchronize()
    check_map(from_dev(dx), orc.conv3x3_backward(np.zeros_like(dyh), wh, dyh, 1)[0], 1, "input gradient", max(1, 128 // W))
    dz = from_dev(dx) * (maskh > 0)
    dxx_ref, dg_ref, db_ref = orc.bn_backward(bxh, mbd.double().cpu().numpy(), isbd.double().cpu().numpy(), gh, dz)
    scale = float(np.sqrt(np.mean(dz ** 2)) * np.sqrt(B * H * W))
    assert np.max(np.abs(db.cpu().numpy() - db_ref)) < 2e-5 * scale and np.max(np.abs(dg.cpu().numpy() - dg_ref)) < 4e-5 * scale
    assert rel(from_dev(dxx), dxx_ref) < TOL[1]
