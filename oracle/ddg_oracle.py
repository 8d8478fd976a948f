"""ctypes binding of the CPU oracle (oracle/ddg_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of the
benchmark.  It never imports the CUDA package, and the CUDA package never imports it.

The oracle follows Section 2 (Eq. 1-5), Section 3.1 (Eq. 6-7) and Section 3.3 (Eq. 8-9, Algorithms 1-2)
of the DDG paper; see the header of ddg_oracle.c for the readings taken where the paper is silent.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ddg_oracle.c")
_LIB = os.path.join(_HERE, "libddg_oracle.so")

FC, CONV3X3, BN, RELU, BASIC_BLOCK, GLOBAL_AVGPOOL, BASIC_BLOCK_PROJ = range(7)
SGD, ADAM = 0, 1
USE_CURRENT_WEIGHTS, WARMUP_DECAY, ROUND_BF16, ROUND_FP32 = 1, 2, 4, 8


class _Layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("kind", "c_in", "c_out", "stride", "has_bias", "relu_after")]


def build(force=False):
    """Compile the oracle with gcc (-O2, OpenMP).  Building the checker is not using it."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        L.orc_create.restype = ctypes.c_void_p
        L.orc_create.argtypes = [ctypes.POINTER(_Layer), ctypes.c_int, ip, ctypes.c_int, ctypes.c_int] + \
            [ctypes.c_double] * 6 + [ctypes.c_int] * 6
        L.orc_destroy.argtypes = [ctypes.c_void_p]
        L.orc_param_count.restype = ctypes.c_size_t
        L.orc_param_count.argtypes = [ctypes.c_void_p]
        L.orc_module_param_counts.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_size_t)]
        L.orc_set_weights.argtypes = [ctypes.c_void_p, dp]
        L.orc_get_weights.argtypes = [ctypes.c_void_p, dp]
        L.orc_set_lr.argtypes = [ctypes.c_void_p, ctypes.c_double]
        L.orc_get_grads.restype = ctypes.c_int
        L.orc_get_grads.argtypes = [ctypes.c_void_p, ctypes.c_int, dp]
        L.orc_loss_only.restype = ctypes.c_double
        L.orc_loss_only.argtypes = [ctypes.c_void_p, dp, ip]
        L.orc_step.restype = ctypes.c_double
        L.orc_step.argtypes = [ctypes.c_void_p, dp, ip]
        L.orc_bf16_round.restype = ctypes.c_double
        L.orc_bf16_round.argtypes = [ctypes.c_double]
        _lib = L
    return _lib


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int))


class Oracle:
    """One DDG training run on the CPU.  `layers` is a list of (kind, c_in, c_out, stride, has_bias,
    relu_after) tuples, `split_after` the K-1 layer indices after which a new module starts."""

    def __init__(self, layers, split_after, batch, in_shape, num_classes, opt="sgd", lr=0.01, momentum=0.0,
                 weight_decay=0.0, beta1=0.9, beta2=0.999, eps=1e-8, flags=0):
        L = lib()
        arr = (_Layer * len(layers))(*[_Layer(*map(int, l)) for l in layers])
        K = len(split_after) + 1
        sp = (ctypes.c_int * max(1, K - 1))(*split_after)
        in_c, in_h, in_w = in_shape
        self._h = L.orc_create(arr, len(layers), sp, K, ADAM if opt == "adam" else SGD, lr, momentum,
                               weight_decay, beta1, beta2, eps, batch, in_c, in_h, in_w, num_classes, flags)
        if not self._h:
            raise ValueError("oracle rejected the network specification")
        self.K, self.batch, self.in_shape, self.num_classes = K, batch, (in_c, in_h, in_w), num_classes
        self.n_params = L.orc_param_count(self._h)
        pm = (ctypes.c_size_t * K)()
        L.orc_module_param_counts(self._h, pm)
        self.per_module = [int(v) for v in pm]

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_weights(self, w):
        w, p = _d(w)
        assert w.size == self.n_params
        lib().orc_set_weights(self._h, p)

    def get_weights(self):
        w = np.empty(self.n_params, dtype=np.float64)
        lib().orc_get_weights(self._h, w.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        return w

    def set_lr(self, lr):
        lib().orc_set_lr(self._h, float(lr))

    def step(self, x, y):
        x, xp = _d(x)
        y, yp = _i(y)
        assert x.size == self.batch * int(np.prod(self.in_shape)) and y.size == self.batch
        return lib().orc_step(self._h, xp, yp)

    def loss_only(self, x, y):
        x, xp = _d(x)
        y, yp = _i(y)
        return lib().orc_loss_only(self._h, xp, yp)

    def get_grads(self, k):
        """(sample index s or -1 during warm-up, gradient of module k, 0-based) of the last step."""
        g = np.empty(self.per_module[k], dtype=np.float64)
        s = lib().orc_get_grads(self._h, k, g.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        return s, g


# --- thin wrappers over the per-layer primitives, for the pins ------------------------------------

def _call(name, *args):
    f = getattr(lib(), name)
    f.restype = None
    conv = []
    keep = []
    for a in args:
        if isinstance(a, np.ndarray):
            keep.append(a)
            if a.dtype == np.int32:
                conv.append(a.ctypes.data_as(ctypes.POINTER(ctypes.c_int)))
            else:
                assert a.dtype == np.float64 and a.flags.c_contiguous
                conv.append(a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        elif a is None:
            conv.append(None)
        elif isinstance(a, float):
            conv.append(ctypes.c_double(a))
        else:
            conv.append(ctypes.c_int(int(a)))
    f(*conv)


def fc_forward(x, W, b):
    B, n_in = x.shape
    y = np.empty((B, W.shape[0]))
    _call("orc_fc_forward", B, n_in, W.shape[0], x, W, b, y)
    return y


def fc_backward(x, W, dy, has_bias=True):
    B, n_in = x.shape
    dx, dW = np.empty_like(x), np.empty_like(W)
    db = np.empty(W.shape[0]) if has_bias else None
    _call("orc_fc_backward", B, n_in, W.shape[0], x, W, dy, dx, dW, db)
    return dx, dW, db


def conv3x3_forward(x, w, stride):
    B, Ci, H, Wd = x.shape
    Co = w.shape[0]
    y = np.empty((B, Co, (H - 1) // stride + 1, (Wd - 1) // stride + 1))
    _call("orc_conv3x3_forward", B, Ci, H, Wd, Co, stride, x, w, y)
    return y


def conv3x3_backward(x, w, dy, stride):
    B, Ci, H, Wd = x.shape
    dx, dw = np.empty_like(x), np.empty_like(w)
    _call("orc_conv3x3_backward", B, Ci, H, Wd, w.shape[0], stride, x, w, dy, dx, dw)
    return dx, dw


def conv1x1_forward(x, w, stride):
    B, Ci, H, Wd = x.shape
    y = np.empty((B, w.shape[0], (H - 1) // stride + 1, (Wd - 1) // stride + 1))
    _call("orc_conv1x1_forward", B, Ci, H, Wd, w.shape[0], stride, x, w, y)
    return y


def conv1x1_backward(x, w, dy, stride):
    B, Ci, H, Wd = x.shape
    dx, dw = np.empty_like(x), np.empty_like(w)
    _call("orc_conv1x1_backward", B, Ci, H, Wd, w.shape[0], stride, x, w, dy, dx, dw)
    return dx, dw


def bn_forward(x, gamma, beta):
    B, C = x.shape[:2]
    HW = int(np.prod(x.shape[2:]))
    y, mean, invstd = np.empty_like(x), np.empty(C), np.empty(C)
    _call("orc_bn_forward", B, C, HW, x, gamma, beta, y, mean, invstd)
    return y, mean, invstd


def bn_backward(x, mean, invstd, gamma, dy):
    B, C = x.shape[:2]
    HW = int(np.prod(x.shape[2:]))
    dx, dg, db = np.empty_like(x), np.empty(C), np.empty(C)
    _call("orc_bn_backward", B, C, HW, x, mean, invstd, gamma, dy, dx, dg, db)
    return dx, dg, db


def shortcut_forward(x, c_out, stride):
    B, Ci, H, Wd = x.shape
    y = np.empty((B, c_out, (H - 1) // stride + 1, (Wd - 1) // stride + 1))
    _call("orc_shortcut_forward", B, Ci, H, Wd, c_out, stride, x, y)
    return y


def shortcut_backward(dy, c_in, H, W, stride):
    B, Co = dy.shape[:2]
    dx = np.empty((B, c_in, H, W))
    _call("orc_shortcut_backward", B, c_in, H, W, Co, stride, dy, dx)
    return dx


def avgpool_forward(x):
    B, C = x.shape[:2]
    y = np.empty((B, C))
    _call("orc_avgpool_forward", B, C, int(np.prod(x.shape[2:])), x, y)
    return y


def avgpool_backward(dy, H, W):
    B, C = dy.shape
    dx = np.empty((B, C, H, W))
    _call("orc_avgpool_backward", B, C, H * W, dy, dx)
    return dx


def softmax_ce(z, y):
    B, C = z.shape
    loss = np.empty(1)
    dz = np.empty_like(z)
    _call("orc_softmax_ce", B, C, z, np.ascontiguousarray(y, dtype=np.int32), loss, dz)
    return float(loss[0]), dz


def bf16_round(v):
    return lib().orc_bf16_round(float(v))
