"""fp64 CPU oracle for the per-replica CNN training step (Algorithm 1 of the paper).

TEST INFRASTRUCTURE ONLY: importable from tests, the smoke check and the benchmark's
CPU-baseline leg, never from the product path.  ``oracle.c`` holds the arithmetic (plain
definitions in double); this module marshals numpy arrays to it and ``net.py`` strings the
operations together in the order of Algorithm 1.  Nothing here is shared with the CUDA
library.

Pins (what fixes each function to something other than itself) live in
``tests/test_oracle_pins.py``; every function below is pinned there.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")


def _host_tag() -> str:
    """The library is compiled with -march=native, so its file name carries a hash of this host's CPU flags:
    a copy built on another machine is never loaded."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


_SO = os.path.join(_HERE, f"liboracle-{_host_tag()}.so")


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (OpenMP) into liboracle.so next to it."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


_lib = None
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int32)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_bf16_rne.restype = ctypes.c_double
        _lib.orc_bf16_rne.argtypes = [ctypes.c_double]
        _lib.orc_softmax_xent.restype = ctypes.c_int
    return _lib


def _p(a):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_D)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def out_dim(n_in: int, taps: int, stride: int, pad: int) -> int:
    return (n_in + 2 * pad - taps) // stride + 1


def round_bf16(x):
    """Round-to-nearest-even onto the bfloat16 grid, directly from double."""
    x = _f64(x)
    out = np.empty_like(x)
    lib().orc_round_bf16(_p(x), _p(out), ctypes.c_long(x.size))
    return out


def round_f32(x):
    """Round to the fp32 grid (storage point of logits, BN statistics)."""
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def conv2d_fwd(x, w, stride: int, pad: int):
    """y[n,p,q,k] = sum_{r,s,c} x[n,p*st+r-pad,q*st+s-pad,c] * w[k,r,s,c]; x NHWC, w KRSC."""
    x, w = _f64(x), _f64(w)
    N, H, W, C = x.shape
    K, R, S, C2 = w.shape
    assert C == C2
    y = np.empty((N, out_dim(H, R, stride, pad), out_dim(W, S, stride, pad), K))
    lib().orc_conv2d_fwd(_p(x), _p(w), _p(y), N, H, W, C, K, R, S, stride, pad)
    return y


def conv2d_dgrad(dy, w, x_shape, stride: int, pad: int):
    """Gradient of <conv(x;w), dy> with respect to x (scatter form)."""
    dy, w = _f64(dy), _f64(w)
    N, H, W, C = x_shape
    K, R, S, _ = w.shape
    assert dy.shape == (N, out_dim(H, R, stride, pad), out_dim(W, S, stride, pad), K)
    dx = np.empty((N, H, W, C))
    lib().orc_conv2d_dgrad(_p(dy), _p(w), _p(dx), N, H, W, C, K, R, S, stride, pad)
    return dx


def conv2d_wgrad(dy, x, R: int, S: int, stride: int, pad: int):
    """Gradient of <conv(x;w), dy> with respect to w, laid out KRSC."""
    dy, x = _f64(dy), _f64(x)
    N, H, W, C = x.shape
    K = dy.shape[-1]
    assert dy.shape == (N, out_dim(H, R, stride, pad), out_dim(W, S, stride, pad), K)
    dw = np.empty((K, R, S, C))
    lib().orc_conv2d_wgrad(_p(dy), _p(x), _p(dw), N, H, W, C, K, R, S, stride, pad)
    return dw


def bn_stats(y, eps: float):
    """Per-channel mean, biased variance and 1/sqrt(var+eps) over all leading dims."""
    y = _f64(y)
    C = y.shape[-1]
    M = y.size // C
    mean, var, invstd = np.empty(C), np.empty(C), np.empty(C)
    lib().orc_bn_stats(_p(y), ctypes.c_long(M), C, ctypes.c_double(eps), _p(mean), _p(var), _p(invstd))
    return mean, var, invstd


def bn_relu_apply(y, mean, invstd, gamma, beta, residual, relu: bool):
    """a = relu?(gamma*(y-mean)*invstd + beta (+ residual))."""
    y = _f64(y)
    C = y.shape[-1]
    M = y.size // C
    a = np.empty_like(y)
    res = None if residual is None else _f64(residual)
    lib().orc_bn_relu_apply(_p(y), _p(_f64(mean)), _p(_f64(invstd)), _p(_f64(gamma)), _p(_f64(beta)), _p(res),
                            int(bool(relu)), ctypes.c_long(M), C, _p(a))
    return a


def bn_relu_bwd(da1, da2, y, a, gamma, mean, invstd, relu: bool, want_dres: bool):
    """Backward of bn_relu_apply composed with bn_stats.  Returns dy, dres|None, dgamma, dbeta."""
    da1, y, a = _f64(da1), _f64(y), _f64(a)
    da2 = None if da2 is None else _f64(da2)
    C = y.shape[-1]
    M = y.size // C
    dy = np.empty_like(y)
    dres = np.empty_like(y) if want_dres else None
    dgamma, dbeta = np.empty(C), np.empty(C)
    lib().orc_bn_relu_bwd(_p(da1), _p(da2), _p(y), _p(a), _p(_f64(gamma)), _p(_f64(mean)), _p(_f64(invstd)),
                          int(bool(relu)), ctypes.c_long(M), C, _p(dy), _p(dres), _p(dgamma), _p(dbeta))
    return dy, dres, dgamma, dbeta


def avgpool_fwd(a):
    a = _f64(a)
    N, H, W, C = a.shape
    out = np.empty((N, C))
    lib().orc_avgpool_fwd(_p(a), N, H * W, C, _p(out))
    return out


def avgpool_bwd(dpooled, H: int, W: int):
    dpooled = _f64(dpooled)
    N, C = dpooled.shape
    da = np.empty((N, H, W, C))
    lib().orc_avgpool_bwd(_p(dpooled), N, H * W, C, _p(da))
    return da


def softmax_xent(logits, labels, grad_scale: float):
    """loss = mean_i(lse(z_i) - z_i[y_i]); dz = (softmax - onehot) * grad_scale."""
    z = _f64(logits)
    N, classes = z.shape
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    loss = ctypes.c_double(0.0)
    dz = np.empty_like(z)
    rc = lib().orc_softmax_xent(_p(z), lab.ctypes.data_as(_I), N, classes, ctypes.c_double(grad_scale),
                                ctypes.byref(loss), _p(dz))
    if rc != 0:
        raise ValueError("label outside [0, classes)")
    return loss.value, dz


def sgd_momentum(w, v, g_sum, inv_n: float, lr: float, mu: float, wd: float):
    """g = g_sum*inv_n + wd*w; v = mu*v + g; w = w - lr*v.  Returns new (w, v)."""
    w, v, g = _f64(w).copy(), _f64(v).copy(), _f64(g_sum)
    lib().orc_sgd_momentum(_p(w), _p(v), _p(g), ctypes.c_long(w.size), ctypes.c_double(inv_n),
                           ctypes.c_double(lr), ctypes.c_double(mu), ctypes.c_double(wd))
    return w, v
