"""Thin ctypes binding over the C ABI of libddg.so (include/ddg.h): argument marshalling only.

Every step of the DDG iteration runs inside the library's CUDA kernels.  torch is used by callers for device
memory and streams; this module itself only needs raw pointers (ints) or objects with `.data_ptr()`.
Importing this module loads the library and raises if it has not been built (there is no fallback).
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libddg.so")

if not os.path.exists(LIB_PATH):
    raise ImportError("libddg.so is missing: build it with `python -m paper_1804_10574_b200.build` "
                      "(the DDG step has no CPU or PyTorch fallback)")

_lib = ctypes.CDLL(LIB_PATH)

FP32, BF16 = 0, 1
OPT_SGD, OPT_ADAM = 0, 1
STATUS = {0: "DDG_OK", 1: "DDG_ERR_INVALID_ARG", 2: "DDG_ERR_BAD_SPEC", 3: "DDG_ERR_UNSUPPORTED", 4: "DDG_ERR_OOM",
          5: "DDG_ERR_CUDA", 6: "DDG_ERR_TIMEOUT", 7: "DDG_ERR_STATE"}

# every symbol include/ddg.h declares
EXPORTS = ["ddg_create", "ddg_step", "ddg_step_host", "ddg_set_lr", "ddg_param_count", "ddg_get_weights",
           "ddg_set_weights", "ddg_get_grads", "ddg_get_loss_dev", "ddg_last_step_launches", "ddg_sync",
           "ddg_last_error", "ddg_destroy", "ddg_conv3x3_fwd", "ddg_conv3x3_dgrad",
           "ddg_conv3x3_wgrad_scratch_elems", "ddg_conv3x3_wgrad", "ddg_bn_scratch_elems", "ddg_bn_fwd", "ddg_bn_bwd",
           "ddg_sgd_update", "ddg_tensor_core_path", "ddg_bn_fwd_noalloc",
           "ddg_conv3x3_packed_bytes", "ddg_conv3x3_pack", "ddg_conv3x3_packed", "ddg_bn_bwd_reduce",
           "ddg_debug_wait_timeout", "ddg_debug_shift_stamps", "ddg_conv3x3_fused_scratch_elems",
           "ddg_conv3x3_fwd_stats", "ddg_conv3x3_dgrad_fused", "ddg_conv3x3_s2_dgrad_shortcut",
           "ddg_fc_tensor_core_path", "ddg_fc_fwd", "ddg_fc_bwd", "ddg_state_bytes", "ddg_save_state",
           "ddg_load_state", "ddg_conv1x1_fwd", "ddg_conv1x1_dgrad_add", "ddg_conv1x1_wgrad_scratch_elems",
           "ddg_conv1x1_wgrad", "ddg_conv3x3_bnrelu_fwd_stats", "ddg_conv3x3_fwd_partials",
           "ddg_bn_fwd_partials", "ddg_conv3x3_dgrad_partials", "ddg_bn_bwd_partials", "ddg_conv3x3_fwd_stats_prepared",
           "ddg_piece_times", "ddg_conv3x3_fwd_stats_shared",
           "ddg_step_host_pipelined", "ddg_pipelined_loss", "ddg_conv3x3_dgrad_fused_shared"]


class Layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("kind", "c_in", "c_out", "stride", "has_bias", "relu_after")]


class Opt(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int)] + [(n, ctypes.c_float) for n in
                                           ("lr", "momentum", "weight_decay", "beta1", "beta2", "eps")]


class Cfg(ctypes.Structure):
    _fields_ = [("precision", ctypes.c_int), ("batch", ctypes.c_int), ("in_c", ctypes.c_int), ("in_h", ctypes.c_int),
                ("in_w", ctypes.c_int), ("num_classes", ctypes.c_int), ("seed", ctypes.c_ulonglong),
                ("use_graph", ctypes.c_int), ("debug_checks", ctypes.c_int),
                ("streams", ctypes.POINTER(ctypes.c_void_p)), ("separate_bn_sums", ctypes.c_int),
                ("fuse_bn_apply", ctypes.c_int), ("bn_fold", ctypes.c_int), ("launch_overlap", ctypes.c_int),
                ("time_pieces", ctypes.c_int)]


_vp, _i, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
_lib.ddg_create.argtypes = [ctypes.POINTER(Layer), _i, ctypes.POINTER(_i), _i, ctypes.POINTER(Opt),
                            ctypes.POINTER(Cfg), ctypes.POINTER(_vp)]
_lib.ddg_step.argtypes = [_vp, _vp, _vp, ctypes.POINTER(_f)]
_lib.ddg_step_host.argtypes = [_vp, _vp, _vp, ctypes.POINTER(_f)]
_lib.ddg_set_lr.argtypes = [_vp, _f]
_lib.ddg_step_host_pipelined.argtypes = [_vp, _vp, _vp, ctypes.POINTER(_f)]
_lib.ddg_pipelined_loss.argtypes = [_vp, ctypes.POINTER(_f)]
_lib.ddg_piece_times.argtypes = [_vp, ctypes.POINTER(_f), ctypes.POINTER(_f)]
_lib.ddg_param_count.argtypes = [_vp, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
_lib.ddg_get_weights.argtypes = [_vp, _vp, _sz, _i]
_lib.ddg_set_weights.argtypes = [_vp, _vp, _sz, _i]
_lib.ddg_get_grads.argtypes = [_vp, _i, _vp, _sz, _i, ctypes.POINTER(ctypes.c_long)]
_lib.ddg_get_loss_dev.argtypes = [_vp, ctypes.POINTER(_vp)]
_lib.ddg_last_step_launches.argtypes = [_vp, ctypes.POINTER(ctypes.c_long)]
_lib.ddg_sync.argtypes = [_vp]
_lib.ddg_state_bytes.argtypes = [_vp, ctypes.POINTER(_sz)]
_lib.ddg_save_state.argtypes = [_vp, _vp, _sz]
_lib.ddg_load_state.argtypes = [_vp, _vp, _sz]
_lib.ddg_debug_wait_timeout.argtypes = [_vp, ctypes.c_uint]
_lib.ddg_debug_shift_stamps.argtypes = [_vp, _i, ctypes.c_long]
_lib.ddg_last_error.argtypes = [_vp]
_lib.ddg_last_error.restype = ctypes.c_char_p
_lib.ddg_destroy.argtypes = [_vp]
_lib.ddg_destroy.restype = None
_lib.ddg_conv3x3_fwd.argtypes = [_i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_conv3x3_dgrad.argtypes = [_i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_conv3x3_wgrad_scratch_elems.argtypes = [_i] * 6
_lib.ddg_conv3x3_wgrad_scratch_elems.restype = _sz
_lib.ddg_conv3x3_wgrad.argtypes = [_i, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_bn_scratch_elems.argtypes = [_i]
_lib.ddg_bn_scratch_elems.restype = _sz
_lib.ddg_bn_fwd.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_bn_bwd.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_tensor_core_path.argtypes = [_i] * 6
_lib.ddg_conv3x3_packed_bytes.argtypes = [_i] * 4
_lib.ddg_conv3x3_packed_bytes.restype = _sz
_lib.ddg_conv3x3_pack.argtypes = [_vp, _vp, _i, _vp]
_lib.ddg_conv3x3_packed.argtypes = [_i, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_conv3x3_fused_scratch_elems.argtypes = [_i] * 4
_lib.ddg_conv3x3_fused_scratch_elems.restype = _sz
_lib.ddg_conv3x3_fwd_stats.argtypes = [_vp] * 7 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_fwd_stats_prepared.argtypes = [_vp] * 7 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_fwd_stats_shared.argtypes = [_vp] * 7 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_fwd_partials.argtypes = [_vp] * 5 + [ctypes.POINTER(_i)] + [_i] * 4 + [_vp]
_lib.ddg_bn_fwd_partials.argtypes = [_vp] * 6 + [_i, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_conv3x3_dgrad_partials.argtypes = [_vp] * 11 + [ctypes.POINTER(_i)] + [_i] * 4 + [_vp]
_lib.ddg_bn_bwd_partials.argtypes = [_vp] * 10 + [_i] + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_bnrelu_fwd_stats.argtypes = [_vp] * 13 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_dgrad_fused.argtypes = [_vp] * 13 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_dgrad_fused_shared.argtypes = [_vp] * 13 + [_i] * 4 + [_vp]
_lib.ddg_conv3x3_s2_dgrad_shortcut.argtypes = [_vp] * 5 + [_i] * 4 + [_vp]
_lib.ddg_conv1x1_fwd.argtypes = [_i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_conv1x1_dgrad_add.argtypes = [_i, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_conv1x1_wgrad_scratch_elems.argtypes = [_i, _i]
_lib.ddg_conv1x1_wgrad_scratch_elems.restype = _sz
_lib.ddg_conv1x1_wgrad.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp]
_lib.ddg_fc_tensor_core_path.argtypes = [_i] * 3
_lib.ddg_fc_fwd.argtypes = [_i, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]
_lib.ddg_fc_bwd.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]
_lib.ddg_bn_fwd_noalloc.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_bn_bwd_reduce.argtypes = [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]
_lib.ddg_sgd_update.argtypes = [_i, _vp, _vp, _vp, _vp, _sz, _f, _f, _f, _vp]


class DdgError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS.get(status, status), message))
        self.status = status


def _ptr(a):
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if hasattr(a, "data_ptr"):
        return a.data_ptr()
    if hasattr(a, "ctypes"):
        return a.ctypes.data
    raise TypeError("expected an address, a torch tensor or a numpy array")


def lib():
    return _lib


class Ddg:
    """ddg_create / ddg_step / ddg_get_weights ... with the same names as the C ABI (without the prefix)."""

    def __init__(self, layers, split_after, batch, in_shape, num_classes, precision="fp32", opt="sgd", lr=0.01,
                 momentum=0.0, weight_decay=0.0, beta1=0.9, beta2=0.999, eps=1e-8, seed=0, use_graph=False,
                 debug_checks=False, streams=None, separate_bn_sums=False, fuse_bn_apply=0, bn_fold=0,
                 launch_overlap=0, time_pieces=False):
        arr = (Layer * len(layers))(*[Layer(*map(int, l)) for l in layers])
        K = len(split_after) + 1
        sp = (ctypes.c_int * max(1, K - 1))(*split_after)
        o = Opt(OPT_ADAM if opt == "adam" else OPT_SGD, lr, momentum, weight_decay, beta1, beta2, eps)
        st = None
        if streams is not None:
            assert len(streams) == K
            st = (ctypes.c_void_p * K)(*[int(s) for s in streams])
        cfg = Cfg(BF16 if precision == "bf16" else FP32, batch, in_shape[0], in_shape[1], in_shape[2], num_classes,
                  seed, int(use_graph), int(debug_checks), st, int(separate_bn_sums), int(fuse_bn_apply), int(bn_fold),
                  int(launch_overlap), int(time_pieces))
        h = ctypes.c_void_p()
        rc = _lib.ddg_create(arr, len(layers), sp, K, ctypes.byref(o), ctypes.byref(cfg), ctypes.byref(h))
        if rc != 0:
            raise DdgError(rc, (_lib.ddg_last_error(None) or b"").decode())
        self._h = h
        self.K, self.batch = K, batch
        n = ctypes.c_size_t()
        pm = (ctypes.c_size_t * K)()
        self._check(_lib.ddg_param_count(self._h, ctypes.byref(n), pm))
        self.n_params = n.value
        self.per_module = [int(v) for v in pm]

    def _check(self, rc):
        if rc != 0:
            raise DdgError(rc, (_lib.ddg_last_error(self._h) or b"").decode())

    def destroy(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.ddg_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def step(self, x_dev, y_dev, want_loss=True):
        loss = ctypes.c_float()
        self._check(_lib.ddg_step(self._h, _ptr(x_dev), _ptr(y_dev), ctypes.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def step_host(self, x_host, y_host, want_loss=True):
        loss = ctypes.c_float()
        self._check(_lib.ddg_step_host(self._h, _ptr(x_host), _ptr(y_host), ctypes.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def step_host_pipelined(self, x_host, y_host):
        """Enqueues the iteration; returns the loss of the PREVIOUS iteration (NaN at the first call)."""
        loss = ctypes.c_float()
        self._check(_lib.ddg_step_host_pipelined(self._h, _ptr(x_host), _ptr(y_host), ctypes.byref(loss)))
        return loss.value

    def pipelined_loss(self):
        loss = ctypes.c_float()
        self._check(_lib.ddg_pipelined_loss(self._h, ctypes.byref(loss)))
        return loss.value

    def set_lr(self, lr):
        self._check(_lib.ddg_set_lr(self._h, lr))

    def get_weights(self, dst, on_device=False):
        self._check(_lib.ddg_get_weights(self._h, _ptr(dst), self.n_params, int(on_device)))
        return dst

    def set_weights(self, src, on_device=False):
        self._check(_lib.ddg_set_weights(self._h, _ptr(src), self.n_params, int(on_device)))

    def get_grads(self, k, dst, on_device=False):
        s = ctypes.c_long()
        self._check(_lib.ddg_get_grads(self._h, k, _ptr(dst), self.per_module[k], int(on_device), ctypes.byref(s)))
        return s.value

    def get_loss_dev(self):
        p = ctypes.c_void_p()
        self._check(_lib.ddg_get_loss_dev(self._h, ctypes.byref(p)))
        return p.value

    def last_step_launches(self):
        n = ctypes.c_long()
        self._check(_lib.ddg_last_step_launches(self._h, ctypes.byref(n)))
        return n.value

    def piece_times(self):
        """(forward ms per module, backward + update ms per module) of the last iteration; needs time_pieces."""
        f, b = (ctypes.c_float * self.K)(), (ctypes.c_float * self.K)()
        self._check(_lib.ddg_piece_times(self._h, f, b))
        return list(f), list(b)

    def sync(self):
        self._check(_lib.ddg_sync(self._h))

    def state_bytes(self):
        n = ctypes.c_size_t()
        self._check(_lib.ddg_state_bytes(self._h, ctypes.byref(n)))
        return n.value

    def save_state(self, dst_host):
        """dst_host: a writable host buffer (numpy uint8 array) of state_bytes() bytes."""
        self._check(_lib.ddg_save_state(self._h, _ptr(dst_host), dst_host.nbytes))
        return dst_host

    def load_state(self, src_host):
        self._check(_lib.ddg_load_state(self._h, _ptr(src_host), src_host.nbytes))

    def debug_wait_timeout(self, polls):
        self._check(_lib.ddg_debug_wait_timeout(self._h, polls))

    def debug_shift_stamps(self, k, delta):
        self._check(_lib.ddg_debug_shift_stamps(self._h, k, delta))


def _ok(rc):
    if rc != 0:
        raise DdgError(rc, (_lib.ddg_last_error(None) or b"kernel entry point failed").decode())


def tensor_core_path(B, H, W, Cin, Cout, stride):
    return _lib.ddg_tensor_core_path(B, H, W, Cin, Cout, stride)


def conv3x3_packed_bytes(B, H, W, C):
    return _lib.ddg_conv3x3_packed_bytes(B, H, W, C)


def conv3x3_pack(w, packed, C, stream=None):
    _ok(_lib.ddg_conv3x3_pack(_ptr(w), _ptr(packed), C, stream))


def conv3x3_packed(dgrad, src, w, packed, dst, B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_packed(int(dgrad), _ptr(src), _ptr(w), _ptr(packed), _ptr(dst), B, H, W, C, stream))


def conv3x3_fused_scratch_elems(B, H, W, C):
    return _lib.ddg_conv3x3_fused_scratch_elems(B, H, W, C)


def conv3x3_fwd_stats(x, w, packed, y, mean, invstd, scratch, B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_fwd_stats(_ptr(x), _ptr(w), _ptr(packed), _ptr(y), _ptr(mean), _ptr(invstd), _ptr(scratch),
                                   B, H, W, C, stream))


def conv3x3_fwd_stats_prepared(x, w, packed, y, mean, invstd, scratch, B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_fwd_stats_prepared(_ptr(x), _ptr(w), _ptr(packed), _ptr(y), _ptr(mean), _ptr(invstd),
                                            _ptr(scratch), B, H, W, C, stream))


def conv3x3_fwd_stats_shared(x, w, packed, y, mean, invstd, scratch, B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_fwd_stats_shared(_ptr(x), _ptr(w), _ptr(packed), _ptr(y), _ptr(mean), _ptr(invstd),
                                         _ptr(scratch), B, H, W, C, stream))


def conv3x3_fwd_partials(x, w, packed, y, part, B, H, W, C, stream=None):
    """Returns the number of partial rows the launch left in `part`."""
    n = ctypes.c_int()
    _ok(_lib.ddg_conv3x3_fwd_partials(_ptr(x), _ptr(w), _ptr(packed), _ptr(y), _ptr(part), ctypes.byref(n), B, H, W, C, stream))
    return n.value


def bn_fwd_partials(y, gamma, beta, res, out, part, n_part, mean, invstd, B, HW, C, relu, stream=None):
    _ok(_lib.ddg_bn_fwd_partials(_ptr(y), _ptr(gamma), _ptr(beta), _ptr(res), _ptr(out), _ptr(part), n_part, _ptr(mean),
                                 _ptr(invstd), B, HW, C, int(relu), stream))


def conv3x3_dgrad_partials(dy, w, packed, dx, res_dout, res_out, bn_mask, bn_x, bn_mean, bn_invstd, part, B, H, W, C,
                           stream=None):
    n = ctypes.c_int()
    _ok(_lib.ddg_conv3x3_dgrad_partials(_ptr(dy), _ptr(w), _ptr(packed), _ptr(dx), _ptr(res_dout), _ptr(res_out),
                                        _ptr(bn_mask), _ptr(bn_x), _ptr(bn_mean), _ptr(bn_invstd), _ptr(part),
                                        ctypes.byref(n), B, H, W, C, stream))
    return n.value


def bn_bwd_partials(dout, out, x, gamma, mean, invstd, dx, dgamma, dbeta, part, n_part, B, HW, C, relu, stream=None):
    _ok(_lib.ddg_bn_bwd_partials(_ptr(dout), _ptr(out), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(invstd), _ptr(dx),
                                 _ptr(dgamma), _ptr(dbeta), _ptr(part), n_part, B, HW, C, int(relu), stream))


def conv3x3_bnrelu_fwd_stats(x, res, gamma, beta, mean_in, invstd_in, a_out, w, packed, y, mean, invstd, scratch, B, H, W,
                             C, stream=None):
    _ok(_lib.ddg_conv3x3_bnrelu_fwd_stats(_ptr(x), _ptr(res), _ptr(gamma), _ptr(beta), _ptr(mean_in), _ptr(invstd_in), _ptr(a_out),
                                          _ptr(w), _ptr(packed), _ptr(y), _ptr(mean), _ptr(invstd), _ptr(scratch), B, H, W, C,
                                          stream))


def conv3x3_dgrad_fused(dy, w, packed, dx, res_dout, res_out, bn_mask, bn_x, bn_mean, bn_invstd, dbeta, dgamma, scratch,
                        B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_dgrad_fused(_ptr(dy), _ptr(w), _ptr(packed), _ptr(dx), _ptr(res_dout), _ptr(res_out),
                                     _ptr(bn_mask), _ptr(bn_x), _ptr(bn_mean), _ptr(bn_invstd), _ptr(dbeta), _ptr(dgamma),
                                     _ptr(scratch), B, H, W, C, stream))


def conv3x3_dgrad_fused_shared(dy, w, packed, dx, res_dout, res_out, bn_mask, bn_x, bn_mean, bn_invstd, dbeta, dgamma,
                               scratch, B, H, W, C, stream=None):
    _ok(_lib.ddg_conv3x3_dgrad_fused_shared(_ptr(dy), _ptr(w), _ptr(packed), _ptr(dx), _ptr(res_dout), _ptr(res_out),
                                            _ptr(bn_mask), _ptr(bn_x), _ptr(bn_mean), _ptr(bn_invstd), _ptr(dbeta),
                                            _ptr(dgamma), _ptr(scratch), B, H, W, C, stream))


def conv3x3_s2_dgrad_shortcut(dy, w, dx, res_dout, res_out, B, H, W, Cin, stream=None):
    _ok(_lib.ddg_conv3x3_s2_dgrad_shortcut(_ptr(dy), _ptr(w), _ptr(dx), _ptr(res_dout), _ptr(res_out), B, H, W, Cin,
                                           stream))


def conv3x3_fwd(prec, x, w, y, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv3x3_fwd(prec, _ptr(x), _ptr(w), _ptr(y), B, H, W, Cin, Cout, stride, stream))


def conv3x3_dgrad(prec, dy, w, dx, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv3x3_dgrad(prec, _ptr(dy), _ptr(w), _ptr(dx), B, H, W, Cin, Cout, stride, stream))


def conv3x3_wgrad_scratch_elems(B, H, W, Cin, Cout, stride):
    return _lib.ddg_conv3x3_wgrad_scratch_elems(B, H, W, Cin, Cout, stride)


def conv3x3_wgrad(prec, x, dy, dw, scratch, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv3x3_wgrad(prec, _ptr(x), _ptr(dy), _ptr(dw), _ptr(scratch), B, H, W, Cin, Cout, stride, stream))


def conv1x1_fwd(prec, x, w, y, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv1x1_fwd(prec, _ptr(x), _ptr(w), _ptr(y), B, H, W, Cin, Cout, stride, stream))


def conv1x1_dgrad_add(prec, dout, out, w, dx, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv1x1_dgrad_add(prec, _ptr(dout), _ptr(out), _ptr(w), _ptr(dx), B, H, W, Cin, Cout, stride, stream))


def conv1x1_wgrad_scratch_elems(Cin, Cout):
    return _lib.ddg_conv1x1_wgrad_scratch_elems(Cin, Cout)


def conv1x1_wgrad(prec, x, dout, out, dw, scratch, B, H, W, Cin, Cout, stride, stream=None):
    _ok(_lib.ddg_conv1x1_wgrad(prec, _ptr(x), _ptr(dout), _ptr(out), _ptr(dw), _ptr(scratch), B, H, W, Cin, Cout, stride,
                               stream))


def fc_tensor_core_path(B, n_in, n_out):
    return _lib.ddg_fc_tensor_core_path(B, n_in, n_out)


def fc_fwd(prec, x, W, bias, y, B, n_in, n_out, relu, out_f32, stream=None):
    _ok(_lib.ddg_fc_fwd(prec, _ptr(x), _ptr(W), _ptr(bias), _ptr(y), B, n_in, n_out, int(relu), int(out_f32), stream))


def fc_bwd(prec, x, W, y, dy, dx, dW, db, B, n_in, n_out, relu, out_f32, stream=None):
    _ok(_lib.ddg_fc_bwd(prec, _ptr(x), _ptr(W), _ptr(y), _ptr(dy), _ptr(dx), _ptr(dW), _ptr(db), B, n_in, n_out,
                        int(relu), int(out_f32), stream))


def bn_scratch_elems(C):
    return _lib.ddg_bn_scratch_elems(C)


def bn_fwd(prec, x, gamma, beta, res, y, mean, invstd, scratch, B, HW, C, relu, stream=None):
    _ok(_lib.ddg_bn_fwd(prec, _ptr(x), _ptr(gamma), _ptr(beta), _ptr(res), _ptr(y), _ptr(mean), _ptr(invstd),
                        _ptr(scratch), B, HW, C, int(relu), stream))


def bn_fwd_noalloc(prec, x, gamma, beta, res, y, mean, invstd, B, HW, C, relu, stream=None):
    """ddg_bn_fwd with the scratch inside the library (C <= 64): allocates nothing.  Returns the status code."""
    return _lib.ddg_bn_fwd_noalloc(prec, _ptr(x), _ptr(gamma), _ptr(beta), _ptr(res), _ptr(y), _ptr(mean),
                                   _ptr(invstd), B, HW, C, int(relu), stream)


def bn_bwd(prec, dout, out, x, gamma, mean, invstd, dx, dgamma, dbeta, scratch, B, HW, C, relu, stream=None):
    _ok(_lib.ddg_bn_bwd(prec, _ptr(dout), _ptr(out), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(invstd), _ptr(dx),
                        _ptr(dgamma), _ptr(dbeta), _ptr(scratch), B, HW, C, int(relu), stream))


def bn_bwd_reduce(prec, dout, out, x, mean, invstd, dgamma, dbeta, scratch, B, HW, C, relu, stream=None):
    _ok(_lib.ddg_bn_bwd_reduce(prec, _ptr(dout), _ptr(out), _ptr(x), _ptr(mean), _ptr(invstd), _ptr(dgamma), _ptr(dbeta),
                               _ptr(scratch), B, HW, C, int(relu), stream))


def sgd_update(prec, w, v, g, w_version, n, lr, momentum, weight_decay, stream=None):
    _ok(_lib.ddg_sgd_update(prec, _ptr(w), _ptr(v), _ptr(g), _ptr(w_version), n, lr, momentum, weight_decay, stream))
