"""Seeded synthetic workloads: network descriptions, parameters, images, labels.

This module serves both the CUDA library's tests/benchmark and the CPU oracle, and holds
none of the method's arithmetic: it only draws random numbers, snaps them to the bf16 grid
(a library cast) and lists layer shapes.  The images stand in for CIFAR-100-shaped data
(32x32x3, 100 classes; per-channel normalised pixels are roughly zero-mean, unit-variance,
hence N(0,1)).

A network is a list of layer dicts.  Tensor 0 is the image batch; layer i writes tensor i+1.
  {"kind": "conv", "src": t, "C", "K", "R", "stride", "pad", "H", "W"}      3x3 / 1x1 convolution
  {"kind": "bn",   "src": t, "res": t | -1, "relu": bool, "C", "H", "W"}    BatchNorm (+residual)(+ReLU)
  {"kind": "avgpool", "src": t, "C", "H", "W"}                              global average pool
  {"kind": "fc",   "src": t, "C", "K"}                                      fully connected + bias
  {"kind": "xent", "src": t, "K"}                                           softmax cross-entropy
H, W are the spatial sizes of the layer's *input*.
"""
from __future__ import annotations

import zlib

import numpy as np
import torch


def rng_for(seed: int, name: str) -> np.random.Generator:
    """One independent Philox stream per (seed, tensor name)."""
    ss = np.random.SeedSequence([int(seed), zlib.crc32(name.encode())])
    return np.random.Generator(np.random.Philox(ss))


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """fp32 array whose every value is exactly representable in bf16 (library RNE cast)."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def normal_bf16(seed: int, name: str, shape, std: float = 1.0) -> np.ndarray:
    return to_bf16_grid(rng_for(seed, name).standard_normal(shape) * std)


def labels_uniform(seed: int, name: str, n: int, classes: int) -> np.ndarray:
    return rng_for(seed, name).integers(0, classes, size=n, dtype=np.int32)


# ------------------------------------------------------------------------------------------
# network descriptions
# ------------------------------------------------------------------------------------------
def _conv(spec, src, C, K, R, stride, H, W, name):
    spec.append(dict(kind="conv", src=src, C=C, K=K, R=R, stride=stride, pad=(R - 1) // 2, H=H, W=W, name=name))
    return len(spec)


def _bn(spec, src, C, H, W, relu, res=-1, name=""):
    spec.append(dict(kind="bn", src=src, res=res, relu=bool(relu), C=C, H=H, W=W, name=name))
    return len(spec)


def _basic_block(spec, t_in, C, K, stride, H, W, name):
    """a1 = relu(bn(conv3x3(x))); out = relu(bn(conv3x3(a1)) + shortcut(x)).
    shortcut = identity, or bn(conv1x1 stride) without ReLU when the shape changes."""
    Ho, Wo = (H + 2 - 3) // stride + 1, (W + 2 - 3) // stride + 1
    t = _conv(spec, t_in, C, K, 3, stride, H, W, name + "c1")
    t = _bn(spec, t, K, Ho, Wo, True, name=name + "bn1")
    if stride != 1 or C != K:
        ts = _conv(spec, t_in, C, K, 1, stride, H, W, name + "sc")
        ts = _bn(spec, ts, K, Ho, Wo, False, name=name + "scbn")
    else:
        ts = t_in
    t = _conv(spec, t, K, K, 3, 1, Ho, Wo, name + "c2")
    t = _bn(spec, t, K, Ho, Wo, True, res=ts, name=name + "bn2")
    return t, Ho, Wo


def _bottleneck_block(spec, t_in, C, width, stride, H, W, name, expansion=4):
    """a1 = relu(bn(conv1x1(x))); a2 = relu(bn(conv3x3 stride(a1))); out = relu(bn(conv1x1(a2)) + shortcut(x)),
    the last 1x1 widening to expansion*width channels.  shortcut as in the basic block."""
    K = expansion * width
    Ho, Wo = (H + 2 - 3) // stride + 1, (W + 2 - 3) // stride + 1
    t = _conv(spec, t_in, C, width, 1, 1, H, W, name + "c1")
    t = _bn(spec, t, width, H, W, True, name=name + "bn1")
    if stride != 1 or C != K:
        ts = _conv(spec, t_in, C, K, 1, stride, H, W, name + "sc")
        ts = _bn(spec, ts, K, Ho, Wo, False, name=name + "scbn")
    else:
        ts = t_in
    t = _conv(spec, t, width, width, 3, stride, H, W, name + "c2")
    t = _bn(spec, t, width, Ho, Wo, True, name=name + "bn2")
    t = _conv(spec, t, width, K, 1, 1, Ho, Wo, name + "c3")
    t = _bn(spec, t, K, Ho, Wo, True, res=ts, name=name + "bn3")
    return t, Ho, Wo


def _head(spec, t, C, H, W, classes):
    spec.append(dict(kind="avgpool", src=t, C=C, H=H, W=W, name="pool"))
    spec.append(dict(kind="fc", src=len(spec), C=C, K=classes, name="fc"))
    spec.append(dict(kind="xent", src=len(spec), K=classes, name="xent"))


def residual_net_spec(stem_width, widths, strides, blocks_per_stage, classes=100, image_hw=32, image_c=3):
    spec = []
    H = W = image_hw
    t = _conv(spec, 0, image_c, stem_width, 3, 1, H, W, "stem")
    t = _bn(spec, t, stem_width, H, W, True, name="stembn")
    C = stem_width
    for si, (K, st) in enumerate(zip(widths, strides), 1):
        for b in range(blocks_per_stage):
            t, H, W = _basic_block(spec, t, C, K, st if b == 0 else 1, H, W, f"s{si}b{b + 1}")
            C = K
    _head(spec, t, C, H, W, classes)
    return spec


def bottleneck_net_spec(stem_width, widths, strides, blocks, classes=100, image_hw=32, image_c=3, expansion=4):
    spec = []
    H = W = image_hw
    t = _conv(spec, 0, image_c, stem_width, 3, 1, H, W, "stem")
    t = _bn(spec, t, stem_width, H, W, True, name="stembn")
    C = stem_width
    for si, (width, st, nb) in enumerate(zip(widths, strides, blocks), 1):
        for b in range(nb):
            t, H, W = _bottleneck_block(spec, t, C, width, st if b == 0 else 1, H, W, f"s{si}b{b + 1}", expansion)
            C = expansion * width
    _head(spec, t, C, H, W, classes)
    return spec


def resnet18_spec(classes=100):
    """ResNet-18-shaped CIFAR net: stem 3->64, stages 64/128/256/512 x 2 basic blocks."""
    return residual_net_spec(64, (64, 128, 256, 512), (1, 2, 2, 2), 2, classes)


def wrn28_10_spec(classes=100):
    """Wide-ResNet-28-10-shaped net: stem 3->16, stages 160/320/640 x 4 basic blocks."""
    return residual_net_spec(16, (160, 320, 640), (1, 2, 2), 4, classes)


def resnet50_spec(classes=100):
    """ResNet-50-shaped CIFAR net (the paper's convolutional workload, Section IV-A, at CIFAR resolution):
    stem 3->64, stages of 3/4/6/3 bottleneck blocks with widths 64/128/256/512 (outputs 256..2048)."""
    return bottleneck_net_spec(64, (64, 128, 256, 512), (1, 2, 2, 2), (3, 4, 6, 3), classes)


def tiny_bottleneck_spec(classes=10, hw=8, c=16, width=16):
    """Small bottleneck net: one projection block at stride 1, one identity block, one stride-2 block."""
    return bottleneck_net_spec(width, (width, 2 * width), (1, 2), (2, 1), classes, image_hw=hw, image_c=c, expansion=2)


def tiny_net_spec(classes=10, hw=8, c=16, width=16, width2=32):
    """Small net with every layer kind (identity block, projection block with stride 2)."""
    return residual_net_spec(width, (width, width2), (1, 2), 1, classes, image_hw=hw, image_c=c)


# ------------------------------------------------------------------------------------------
# parameters and batches
# ------------------------------------------------------------------------------------------
def init_params(spec, seed: int = 0) -> dict:
    """fp32 master parameters: Kaiming-normal (fan_in) conv/FC weights, gamma=1, beta=0, bias=0."""
    params = {}
    for i, L in enumerate(spec):
        if L["kind"] == "conv":
            fan_in = L["R"] * L["R"] * L["C"]
            w = rng_for(seed, f"w{i}").standard_normal((L["K"], L["R"], L["R"], L["C"])) * np.sqrt(2.0 / fan_in)
            params[f"w{i}"] = w.astype(np.float32)
        elif L["kind"] == "fc":
            w = rng_for(seed, f"w{i}").standard_normal((L["K"], L["C"])) * np.sqrt(2.0 / L["C"])
            params[f"w{i}"] = w.astype(np.float32)
            params[f"b{i}"] = np.zeros(L["K"], np.float32)
        elif L["kind"] == "bn":
            params[f"gamma{i}"] = np.ones(L["C"], np.float32)
            params[f"beta{i}"] = np.zeros(L["C"], np.float32)
    return params


def perturb_bn_params(params: dict, seed: int = 0) -> dict:
    """Non-trivial gamma/beta/bias (so tests exercise them); values stay fp32."""
    out = dict(params)
    for k, v in params.items():
        if k.startswith("gamma"):
            out[k] = (1.0 + 0.25 * rng_for(seed, k).standard_normal(v.shape)).astype(np.float32)
        elif k.startswith("beta") or k.startswith("b"):
            out[k] = (0.1 * rng_for(seed, k).standard_normal(v.shape)).astype(np.float32)
    return out


def image_batch(seed: int, n: int, hw: int = 32, c: int = 3, classes: int = 100, tag: str = ""):
    """(images fp32-on-bf16-grid [n,hw,hw,c], labels int32 [n])."""
    return normal_bf16(seed, "images" + tag, (n, hw, hw, c)), labels_uniform(seed, "labels" + tag, n, classes)


def conv_problem(seed: int, N, H, W, C, K, R, stride):
    """x ~ N(0,1), Kaiming-normal w, upstream gradient ~ N(0,1); all on the bf16 grid."""
    pad = (R - 1) // 2
    P, Q = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    x = normal_bf16(seed, "x", (N, H, W, C))
    w = normal_bf16(seed, "w", (K, R, R, C), std=float(np.sqrt(2.0 / (R * R * C))))
    g = normal_bf16(seed, "g", (N, P, Q, K))
    return x, w, g
