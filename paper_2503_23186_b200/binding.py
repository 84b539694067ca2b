"""ctypes binding of libb2c.so (the C ABI declared in include/b2c.h).

Argument marshalling only: torch supplies device memory and the current stream, every
computation happens inside the library's kernels.  There is no fallback: if the shared
library has not been built, ``lib()`` raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_double, c_float, c_int, c_int32, c_long, c_longlong, c_size_t, c_uint, c_void_p

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
SO_PATH = os.path.join(_HERE, "libb2c.so")

STATUS_NAMES = {0: "B2C_OK", 1: "B2C_ERR_INVALID_ARG", 2: "B2C_ERR_UNSUPPORTED_SHAPE", 3: "B2C_ERR_MISALIGNED",
                4: "B2C_ERR_WORKSPACE_TOO_SMALL", 5: "B2C_ERR_CUDA", 6: "B2C_ERR_ARCH", 7: "B2C_ERR_DEVICE_TIMEOUT",
                8: "B2C_ERR_BAD_LABEL"}
LAYER_KINDS = {"conv": 0, "bn": 1, "avgpool": 2, "fc": 3, "xent": 4}

# every symbol include/b2c.h declares
EXPORTS = [
    "b2c_create", "b2c_destroy", "b2c_status_string", "b2c_get_device_status", "b2c_set_spin_limit", "b2c_set_stall_counters",
    "b2c_conv2d_workspace_bytes", "b2c_conv2d_fwd", "b2c_bn_relu_fwd", "b2c_avgpool_fwd", "b2c_avgpool_bwd", "b2c_pad_channels",
    "b2c_softmax_xent_fwd_bwd", "b2c_bn_relu_bwd_workspace_bytes", "b2c_bn_relu_bwd", "b2c_bn_relu_bwd_static",
    "b2c_bn_relu_bwd_groups_workspace_bytes", "b2c_bn_relu_bwd_groups", "b2c_conv2d_dgrad",
    "b2c_conv2d_wgrad", "b2c_bias_grad", "b2c_grad_accum_sgd_momentum", "b2c_weight_pack_dgrad",
    "b2c_net_create", "b2c_net_create_concurrent", "b2c_net_destroy", "b2c_net_param_count", "b2c_net_param_offset",
    "b2c_net_padded_image_channels", "b2c_net_first_conv_im2col", "b2c_im2col_3x3", "b2c_net_workspace_bytes", "b2c_net_tensor_offset", "b2c_net_bind",
    "b2c_net_sync_weights", "b2c_train_step", "b2c_net_apply_update", "b2c_net_profile_enable", "b2c_net_profile_read",
    "b2c_net_profile_read_layers", "b2c_net_layer_count",
    "b2c_net_weight_layer_count", "b2c_net_weight_range", "b2c_net_refresh_dgrad_weights", "b2c_net_set_buckets", "b2c_net_bucket_wait",
    "b2c_net_running_stats_count", "b2c_net_running_stats_offset", "b2c_net_bind_running_stats",
]
PROF_KINDS = ["conv_fwd", "conv_dgrad", "conv_wgrad", "bn_fwd", "bn_bwd", "other", "update"]


class ConvDesc(Structure):
    _fields_ = [(n, c_int) for n in ("n", "h", "w", "c", "k", "r", "s", "stride", "pad")]


class WeightSeg(Structure):
    _fields_ = [("offset", c_longlong), ("k", c_int), ("rs", c_int), ("c", c_int)]


class LayerDesc(Structure):
    _fields_ = [(n, c_int) for n in ("kind", "src", "res", "relu", "c", "k", "r", "stride", "h", "w")]


class B2CError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(SO_PATH):
            raise RuntimeError(f"{SO_PATH} is missing: build it with `python -m paper_2503_23186_b200.build` "
                               "(there is no CPU or library fallback)")
        L = ctypes.CDLL(SO_PATH)
        L.b2c_status_string.restype = ctypes.c_char_p
        L.b2c_net_param_count.restype = c_size_t
        L.b2c_net_workspace_bytes.restype = c_size_t
        L.b2c_bn_relu_bwd_workspace_bytes.restype = c_size_t
        L.b2c_conv2d_workspace_bytes.restype = c_size_t
        L.b2c_bn_relu_bwd_groups_workspace_bytes.restype = c_size_t
        L.b2c_net_param_offset.restype = c_longlong
        L.b2c_net_tensor_offset.restype = c_longlong
        L.b2c_net_running_stats_count.restype = c_size_t
        L.b2c_net_running_stats_offset.restype = c_longlong
        L.b2c_destroy.restype = None
        L.b2c_net_destroy.restype = None
        L.b2c_set_spin_limit.restype = None
        L.b2c_set_stall_counters.restype = None
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return c_void_p(None)
    if isinstance(t, int):
        return c_void_p(t)
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise B2CError(status, where)


def conv_desc(n, h, w, c, k, r, stride) -> ConvDesc:
    return ConvDesc(n, h, w, c, k, r, r, stride, (r - 1) // 2)


class Context:
    """One per host thread; owns the device status word."""

    def __init__(self, device: int = 0):
        self.handle = c_void_p()
        _check(lib().b2c_create(byref(self.handle), c_int(device)), "b2c_create")

    def close(self):
        if self.handle:
            lib().b2c_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- status
    def device_status(self) -> int:
        return lib().b2c_get_device_status(self.handle, _stream())

    def check_device(self):
        _check(self.device_status(), "device status")

    def set_spin_limit(self, limit: int):
        lib().b2c_set_spin_limit(self.handle, c_uint(limit))

    def set_stall_counters(self, counters):
        """counters: int64 device tensor of 8 words (or None to switch the diagnostics off)."""
        lib().b2c_set_stall_counters(self.handle, _ptr(counters))

    # ---- forward
    def conv2d_fwd(self, d: ConvDesc, x, w_krsc, y, bias=None, ch_stats=None):
        _check(lib().b2c_conv2d_fwd(self.handle, byref(d), _ptr(x), _ptr(w_krsc), _ptr(y), c_int(int(y.dtype == torch.float32)),
                                    _ptr(bias), _ptr(ch_stats), _stream()), "b2c_conv2d_fwd")

    def bn_relu_fwd(self, n, h, w, c, y, ch_stats, stats_ready, gamma, beta, residual, relu, eps, a, save_mean, save_invstd,
                    run_mean=None, run_var=None, momentum=0.1, relu_mask=None):
        _check(lib().b2c_bn_relu_fwd(self.handle, n, h, w, c, _ptr(y), _ptr(ch_stats), c_int(int(stats_ready)), _ptr(gamma), _ptr(beta),
                                     _ptr(residual), c_int(int(relu)), c_float(eps), _ptr(a), _ptr(save_mean), _ptr(save_invstd),
                                     _ptr(run_mean), _ptr(run_var), c_float(momentum), _ptr(relu_mask), _stream()), "b2c_bn_relu_fwd")

    def avgpool_fwd(self, n, hw, c, a, pooled):
        _check(lib().b2c_avgpool_fwd(self.handle, n, hw, c, _ptr(a), _ptr(pooled), _stream()), "b2c_avgpool_fwd")

    def avgpool_bwd(self, n, hw, c, dpooled, da):
        _check(lib().b2c_avgpool_bwd(self.handle, n, hw, c, _ptr(dpooled), _ptr(da), _stream()), "b2c_avgpool_bwd")

    def im2col_3x3(self, n, h, w, c_in, c_out, x, y):
        _check(lib().b2c_im2col_3x3(self.handle, n, h, w, c_in, c_out, _ptr(x), _ptr(y), _stream()), "b2c_im2col_3x3")

    def pad_channels(self, m, c_in, c_out, x, y):
        _check(lib().b2c_pad_channels(self.handle, c_long(m), c_in, c_out, _ptr(x), _ptr(y), _stream()), "b2c_pad_channels")

    # ---- loss
    def softmax_xent_fwd_bwd(self, n, classes, logits, logits_pitch, labels, loss_scale, grad_scale, loss, dlogits, pitch):
        _check(lib().b2c_softmax_xent_fwd_bwd(self.handle, n, classes, _ptr(logits), logits_pitch, _ptr(labels), c_float(loss_scale),
                                              c_float(grad_scale), _ptr(loss), _ptr(dlogits), pitch, _stream()), "b2c_softmax_xent_fwd_bwd")

    # ---- backward
    @staticmethod
    def bn_relu_bwd_workspace_bytes(c) -> int:
        return lib().b2c_bn_relu_bwd_workspace_bytes(c_int(c))

    def bn_relu_bwd(self, n, h, w, c, da1, da2, y, a, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta, acc, ws, relu_mask=None):
        _check(lib().b2c_bn_relu_bwd(self.handle, n, h, w, c, _ptr(da1), _ptr(da2), _ptr(y), _ptr(a), _ptr(gamma), _ptr(save_mean),
                                     _ptr(save_invstd), c_int(int(relu)), _ptr(dy), _ptr(dres), _ptr(dgamma), _ptr(dbeta), c_int(int(acc)),
                                     _ptr(relu_mask), _ptr(ws), c_size_t(ws.numel() * ws.element_size()), _stream()), "b2c_bn_relu_bwd")

    @staticmethod
    def bn_relu_bwd_groups_workspace_bytes(c, groups) -> int:
        return lib().b2c_bn_relu_bwd_groups_workspace_bytes(c_int(c), c_int(groups))

    def bn_relu_bwd_groups(self, groups, rows_per_group, c, da1, da2, y, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta, acc, relu_mask, ws):
        """BatchNorm backward of `groups` statistics groups stored back to back (both passes in one launch, group by group)."""
        _check(lib().b2c_bn_relu_bwd_groups(self.handle, c_int(groups), c_longlong(rows_per_group), c_int(c), _ptr(da1), _ptr(da2), _ptr(y), _ptr(gamma),
                                            _ptr(save_mean), _ptr(save_invstd), c_int(int(relu)), _ptr(dy), _ptr(dres), _ptr(dgamma), _ptr(dbeta),
                                            c_int(int(acc)), _ptr(relu_mask), _ptr(ws), c_size_t(ws.numel() * ws.element_size()), _stream()),
               "b2c_bn_relu_bwd_groups")

    def bn_relu_bwd_static(self, n, h, w, c, da1, da2, y, a, gamma, save_mean, save_invstd, relu, dy, dres, dgamma, dbeta, acc):
        """b2c_bn_relu_bwd without a caller-provided workspace: the accumulators live inside the library, so the
        call allocates nothing (for callers that cannot get device memory of their own; at most 2048 channels;
        calls that overlap on the GPU race on the shared scratch)."""
        _check(lib().b2c_bn_relu_bwd_static(self.handle, n, h, w, c, _ptr(da1), _ptr(da2), _ptr(y), _ptr(a), _ptr(gamma), _ptr(save_mean),
                                            _ptr(save_invstd), c_int(int(relu)), _ptr(dy), _ptr(dres), _ptr(dgamma), _ptr(dbeta),
                                            c_int(int(acc)), _stream()), "b2c_bn_relu_bwd_static")

    def conv2d_dgrad(self, d: ConvDesc, dy, w_crsk_flipped, dx):
        _check(lib().b2c_conv2d_dgrad(self.handle, byref(d), _ptr(dy), _ptr(w_crsk_flipped), _ptr(dx), _stream()), "b2c_conv2d_dgrad")

    def conv2d_wgrad(self, d: ConvDesc, dy, x, dw, accumulate=False):
        _check(lib().b2c_conv2d_wgrad(self.handle, byref(d), _ptr(dy), _ptr(x), _ptr(dw), c_int(int(accumulate)), _stream()), "b2c_conv2d_wgrad")

    def bias_grad(self, m, k, pitch, dz, db, accumulate=False):
        _check(lib().b2c_bias_grad(self.handle, m, k, pitch, _ptr(dz), _ptr(db), c_int(int(accumulate)), _stream()), "b2c_bias_grad")

    # ---- update
    def grad_accum_sgd_momentum(self, count, w, v, g_accum, inv_n_micro, lr, momentum, wd, w_bf16=None, zero_grad=True):
        _check(lib().b2c_grad_accum_sgd_momentum(self.handle, c_size_t(count), _ptr(w), _ptr(v), _ptr(g_accum), c_float(inv_n_micro),
                                                 c_float(lr), c_float(momentum), c_float(wd), _ptr(w_bf16), c_int(int(zero_grad)), _stream()),
               "b2c_grad_accum_sgd_momentum")

    def weight_pack_dgrad(self, segs, src_bf16, dst_bf16):
        arr = (WeightSeg * len(segs))(*[WeightSeg(o, k, rs, c) for (o, k, rs, c) in segs])
        _check(lib().b2c_weight_pack_dgrad(self.handle, arr, len(segs), _ptr(src_bf16), _ptr(dst_bf16), _stream()), "b2c_weight_pack_dgrad")


class Net:
    """A layer list bound to device memory; train_step runs the whole optimiser step."""

    def __init__(self, ctx: Context, spec, micro_batch: int, n_concurrent: int = 1):
        self.ctx, self.spec, self.micro_batch, self.n_concurrent = ctx, spec, micro_batch, n_concurrent
        descs = (LayerDesc * len(spec))()
        for i, L in enumerate(spec):
            descs[i] = LayerDesc(LAYER_KINDS[L["kind"]], L["src"], L.get("res", -1), int(L.get("relu", False)), L.get("C", 0), L.get("K", 0),
                                 L.get("R", 0), L.get("stride", 0), L.get("H", 1), L.get("W", 1))
        self.handle = c_void_p()
        _check(lib().b2c_net_create_concurrent(ctx.handle, descs, len(spec), micro_batch, n_concurrent, byref(self.handle)),
               "b2c_net_create_concurrent")
        self.param_count = lib().b2c_net_param_count(self.handle)
        self.workspace_bytes = lib().b2c_net_workspace_bytes(self.handle)
        self.image_c_pad = lib().b2c_net_padded_image_channels(self.handle)
        self.first_conv_im2col = bool(lib().b2c_net_first_conv_im2col(self.handle))
        dev = torch.device("cuda")
        self.w = torch.zeros(self.param_count, dtype=torch.float32, device=dev)
        self.v = torch.zeros_like(self.w)
        self.g = torch.zeros_like(self.w)
        self.w_bf16 = torch.zeros(self.param_count, dtype=torch.bfloat16, device=dev)
        self.w_dgrad = torch.zeros_like(self.w_bf16)
        self.workspace = torch.zeros(self.workspace_bytes, dtype=torch.uint8, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.bucket_events = None
        _check(lib().b2c_net_bind(self.handle, _ptr(self.w), _ptr(self.v), _ptr(self.g), _ptr(self.w_bf16), _ptr(self.w_dgrad),
                                  _ptr(self.workspace), c_size_t(self.workspace_bytes)), "b2c_net_bind")

    def close(self):
        if self.handle:
            lib().b2c_net_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def param_offset(self, layer: int, which: int) -> int:
        return lib().b2c_net_param_offset(self.handle, layer, which)

    def tensor_offset(self, tensor: int, grad: bool = False, which: int = 0) -> int:
        return lib().b2c_net_tensor_offset(self.handle, tensor, int(grad), which)

    # ---- flat-array <-> per-layer parameter dictionaries (host-side layout bookkeeping)
    def _slots(self):
        """Yield (name, offset, stored_shape, logical_shape as laid out inside the stored array)."""
        for i, L in enumerate(self.spec):
            if L["kind"] == "conv":
                if i == 0 and self.first_conv_im2col:   # [k][r][s][c] taps flattened into rows of the patch-matrix GEMM
                    yield f"w{i}", self.param_offset(i, 0), (L["K"], self.image_c_pad), (L["K"], L["R"] * L["R"] * L["C"])
                    continue
                cpad = -(-L["C"] // 16) * 16
                yield f"w{i}", self.param_offset(i, 0), (L["K"], L["R"], L["R"], cpad), (L["K"], L["R"], L["R"], L["C"])
            elif L["kind"] == "fc":
                kpad = -(-L["K"] // 64) * 64
                yield f"w{i}", self.param_offset(i, 0), (kpad, L["C"]), (L["K"], L["C"])
                yield f"b{i}", self.param_offset(i, 3), (kpad,), (L["K"],)
            elif L["kind"] == "bn":
                yield f"gamma{i}", self.param_offset(i, 1), (L["C"],), (L["C"],)
                yield f"beta{i}", self.param_offset(i, 2), (L["C"],), (L["C"],)

    def _logical_shape(self, name):
        L = self.spec[int(name.lstrip("wbgamet"))]
        if name.startswith("w"):
            return (L["K"], L["R"], L["R"], L["C"]) if L["kind"] == "conv" else (L["K"], L["C"])
        return (L["K"],) if name.startswith("b") and not name.startswith("beta") else (L["C"],)

    def pack(self, params: dict) -> np.ndarray:
        flat = np.zeros(self.param_count, np.float32)
        for name, off, stored, logical in self._slots():
            buf = np.zeros(stored, np.float32)
            buf[tuple(slice(0, s) for s in logical)] = np.asarray(params[name]).reshape(logical)
            flat[off:off + buf.size] = buf.reshape(-1)
        return flat

    def unpack(self, flat) -> dict:
        flat = flat.detach().float().cpu().numpy() if isinstance(flat, torch.Tensor) else np.asarray(flat)
        out = {}
        for name, off, stored, logical in self._slots():
            size = int(np.prod(stored))
            out[name] = flat[off:off + size].reshape(stored)[tuple(slice(0, s) for s in logical)].copy().reshape(self._logical_shape(name))
        return out

    def load_params(self, params: dict, velocity: dict | None = None):
        self.w.copy_(torch.from_numpy(self.pack(params)))
        if velocity is not None:
            self.v.copy_(torch.from_numpy(self.pack(velocity)))
        else:
            self.v.zero_()
        self.g.zero_()
        _check(lib().b2c_net_sync_weights(self.handle, _stream()), "b2c_net_sync_weights")

    def train_step(self, images, labels, n_micro, lr, momentum, wd, update=True):
        """images bf16 [n_micro*micro_batch, H, W, C] and labels int32, both on the device."""
        _check(lib().b2c_train_step(self.handle, _ptr(images), _ptr(labels), c_int(n_micro), c_float(lr), c_float(momentum), c_float(wd),
                                    _ptr(self.loss), c_int(int(update)), _stream()), "b2c_train_step")
        return self.loss

    def apply_update(self, n_avg, lr, momentum, wd):
        _check(lib().b2c_net_apply_update(self.handle, c_int(n_avg), c_float(lr), c_float(momentum), c_float(wd), _stream()), "b2c_net_apply_update")

    # ---- pieces of the update for replicas that shard the optimiser state (data_parallel.dp_train_step_sharded)
    def weight_layer_ranges(self):
        """[(begin, end)] element ranges of the filter banks in the flat arrays, in layer order."""
        out = []
        for i in range(lib().b2c_net_weight_layer_count(self.handle)):
            b, e = c_longlong(), c_longlong()
            _check(lib().b2c_net_weight_range(self.handle, c_int(i), byref(b), byref(e)), "b2c_net_weight_range")
            out.append((b.value, e.value))
        return out

    def enable_running_stats(self, momentum: float = 0.1):
        """Allocates and binds the running statistics (mean 0, variance 1); returns {layer: (mean view, var view)}."""
        n = lib().b2c_net_running_stats_count(self.handle)
        self.running = torch.zeros(max(n, 1), dtype=torch.float32, device="cuda")
        views = {}
        for i, L in enumerate(self.spec):
            if L["kind"] != "bn":
                continue
            off = lib().b2c_net_running_stats_offset(self.handle, c_int(i))
            if off < 0:
                continue
            c = L["C"]
            self.running[off + c:off + 2 * c] = 1.0
            views[i] = (self.running[off:off + c], self.running[off + c:off + 2 * c])
        _check(lib().b2c_net_bind_running_stats(self.handle, _ptr(self.running), c_float(momentum)), "b2c_net_bind_running_stats")
        return views

    def set_buckets(self, buckets):
        """buckets = data_parallel.bucket_plan(...): train_step then records a gradient-ready event per bucket."""
        first = (c_int * len(buckets))(*[b[2] for b in buckets])
        _check(lib().b2c_net_set_buckets(self.handle, c_int(len(buckets)), first), "b2c_net_set_buckets")
        self.bucket_events = list(range(len(buckets))) if buckets else None

    def bucket_wait(self, k, stream):
        """Makes the torch stream `stream` wait until bucket k's gradients of the current step are final."""
        _check(lib().b2c_net_bucket_wait(self.handle, c_int(k), c_void_p(stream.cuda_stream)), "b2c_net_bucket_wait")

    def apply_update_range(self, begin, end, n_avg, lr, momentum, wd):
        """The fused average + SGD-momentum update on elements [begin, end) of the flat arrays only (fp32 master, momentum,
        gradient sum cleared, bf16 copy); begin a multiple of 8."""
        self.ctx.grad_accum_sgd_momentum(end - begin, self.w[begin:end], self.v[begin:end], self.g[begin:end], 1.0 / n_avg, lr, momentum, wd,
                                         self.w_bf16[begin:end], True)

    def refresh_derived_weights(self):
        """Rewrites the data-gradient layout of the bf16 weights from the current bf16 copy."""
        _check(lib().b2c_net_refresh_dgrad_weights(self.handle, _stream()), "b2c_net_refresh_dgrad_weights")

    def profile_enable(self, enable: bool = True):
        _check(lib().b2c_net_profile_enable(self.handle, c_int(int(enable))), "b2c_net_profile_enable")

    def profile_read(self):
        """(ms per kernel family, kernels launched per family) since the last read; synchronises."""
        ms = (c_double * len(PROF_KINDS))()
        n = (c_longlong * len(PROF_KINDS))()
        _check(lib().b2c_net_profile_read(self.handle, ms, n, _stream()), "b2c_net_profile_read")
        return dict(zip(PROF_KINDS, list(ms))), dict(zip(PROF_KINDS, list(n)))

    def profile_read_layers(self):
        """Per layer [forward ms, parameter-gradient ms, data-gradient ms] since the last profile_read (call before it)."""
        n = len(self.spec)
        ms = (c_double * (3 * n))()
        _check(lib().b2c_net_profile_read_layers(self.handle, ms, c_int(n), _stream()), "b2c_net_profile_read_layers")
        return np.array(list(ms)).reshape(n, 3)

    def tensor_view(self, tensor: int, shape, dtype=torch.bfloat16, grad=False, which=0):
        off = self.tensor_offset(tensor, grad, which)
        if off < 0:
            return None
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        return self.workspace[off:off + n].view(dtype).view(*shape)
