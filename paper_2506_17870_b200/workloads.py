"""Seeded synthetic inputs and layer tables for tests and benchmarks.

This module holds NO nesting arithmetic: it only draws random tensors with the shapes, sizes and
value distributions of the paper's ImageNet CNN / ViT workloads (ResNet-18, ResNet-101, ViT-B/16)
and lists their layer shapes.  Both the CPU oracle's tests and the CUDA path's tests read their
inputs from here so that they see the same bytes.  Everything is numpy; callers move it where they
need it.  The one formula here is the plain symmetric per-channel INT8 quantiser of Eq. 1, used to
turn Gaussian fp32 "weights" into int8 inputs.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np

BASE_SEED = 250617870


def rng_for(config: int, index: int = 0) -> np.random.Generator:
    return np.random.default_rng(BASE_SEED + 1000 * config + index)


# --------------------------------------------------------------------------- distributions
def uniform_int8(rng, shape, lo=-128, hi=127) -> np.ndarray:
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int16).astype(np.int8)


def clipped_normal_int8(rng, shape, sigma: float) -> np.ndarray:
    z = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(sigma)
    return np.clip(np.rint(z), -128, 127).astype(np.int8)


def bernoulli_mask(rng, shape, p: float = 0.5) -> np.ndarray:
    return (rng.random(size=shape, dtype=np.float32) < p).astype(np.uint8)


def channel_scales(rng, n: int, lo=1e-3, hi=1e-2) -> np.ndarray:
    return rng.uniform(lo, hi, size=n).astype(np.float32)


def quantize_per_channel(w: np.ndarray, n_bits: int = 8) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1 with one scale per output channel (row): s_j = max|w_j| / (2^(n-1) - 1)."""
    qmax = 2 ** (n_bits - 1) - 1
    w2 = w.reshape(w.shape[0], -1)
    s = np.maximum(np.abs(w2).max(axis=1), 1e-12).astype(np.float32) / np.float32(qmax)
    q = np.clip(np.rint(w2 / s[:, None]), -qmax - 1, qmax).astype(np.int8)
    return q.reshape(w.shape), s


def gaussian_weights_int8(rng, shape, fan_in: int) -> Tuple[np.ndarray, np.ndarray]:
    """Random-init weights ~ N(0, 2 / fan_in), then per-channel INT8 (the CNN configs)."""
    w = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
    return quantize_per_channel(w)


def heavy_tail_weights_int8(rng, shape, sigma=0.02, outlier_p=1e-3, outlier_sigmas=6.0):
    """Gaussian weights with a Bernoulli(outlier_p) share of elements replaced by +-6 sigma (ViT config)."""
    w = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(sigma)
    hit = rng.random(size=shape, dtype=np.float32) < outlier_p
    sign = np.where(rng.random(size=shape, dtype=np.float32) < 0.5, -1.0, 1.0).astype(np.float32)
    w = np.where(hit, sign * np.float32(outlier_sigmas * sigma), w)
    return quantize_per_channel(w)


# --------------------------------------------------------------------------- layer tables
@dataclass(frozen=True)
class ConvLayer:
    name: str
    Cin: int
    H: int
    W: int
    Cout: int
    R: int
    S: int
    stride: int
    pad: int

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def K(self) -> int:
        return self.R * self.S * self.Cin

    @property
    def weights(self) -> int:
        return self.Cout * self.K

    def gemm_view(self, batch: int) -> Tuple[int, int, int]:
        return batch * self.Ho * self.Wo, self.Cout, self.K


def resnet18_layers() -> List[ConvLayer]:
    """20 convolutions + the classifier (as a 1x1 convolution on a 1x1 map), 224x224 input."""
    L = [ConvLayer("conv1", 3, 224, 224, 64, 7, 7, 2, 3)]
    size, cin = 56, 64
    for stage, cout in enumerate((64, 128, 256, 512)):
        for block in range(2):
            stride = 2 if (stage > 0 and block == 0) else 1
            L.append(ConvLayer(f"l{stage+1}b{block}c1", cin, size, size, cout, 3, 3, stride, 1))
            out = size // stride
            L.append(ConvLayer(f"l{stage+1}b{block}c2", cout, out, out, cout, 3, 3, 1, 1))
            if stride != 1 or cin != cout:
                L.append(ConvLayer(f"l{stage+1}b{block}ds", cin, size, size, cout, 1, 1, stride, 0))
            size, cin = out, cout
    L.append(ConvLayer("fc", 512, 1, 1, 1000, 1, 1, 1, 0))
    return L


def resnet101_layers() -> List[ConvLayer]:
    """104 convolutions + classifier; bottlenecks [3, 4, 23, 3] with the stride on the 3x3 convolution."""
    L = [ConvLayer("conv1", 3, 224, 224, 64, 7, 7, 2, 3)]
    size, cin = 56, 64
    for stage, (mid, blocks) in enumerate(((64, 3), (128, 4), (256, 23), (512, 3))):
        for block in range(blocks):
            stride = 2 if (stage > 0 and block == 0) else 1
            cout = 4 * mid
            L.append(ConvLayer(f"l{stage+1}b{block}c1", cin, size, size, mid, 1, 1, 1, 0))
            L.append(ConvLayer(f"l{stage+1}b{block}c2", mid, size, size, mid, 3, 3, stride, 1))
            out = size // stride
            L.append(ConvLayer(f"l{stage+1}b{block}c3", mid, out, out, cout, 1, 1, 1, 0))
            if block == 0:
                L.append(ConvLayer(f"l{stage+1}b{block}ds", cin, size, size, cout, 1, 1, stride, 0))
            size, cin = out, cout
    L.append(ConvLayer("fc", 2048, 1, 1, 1000, 1, 1, 1, 0))
    return L


def vit_b16_linears(blocks: int = 12) -> List[Tuple[str, int, int]]:
    """(name, K, N) of the weight-carrying linears of ViT-B/16: fused qkv, projection, MLP up and down."""
    out = []
    for b in range(blocks):
        out += [(f"b{b}.qkv", 768, 2304), (f"b{b}.proj", 768, 768), (f"b{b}.fc1", 768, 3072), (f"b{b}.fc2", 3072, 768)]
    return out


VIT_TOKENS = 197


# --------------------------------------------------------------------------- the five configurations
def config1(seed_index: int = 0) -> Dict[str, object]:
    """Single linear layer, INT(8|6): W 256x256 uniform int8, X 64x256 clipped N(0, 32)."""
    rng = rng_for(1, seed_index)
    return {
        "n_bits": 8, "h_bits": 6,
        "W": uniform_int8(rng, (256, 256)),
        "w_scale": channel_scales(rng, 256),
        "mask": bernoulli_mask(rng, (256, 256)),
        "X": clipped_normal_int8(rng, (64, 256), 32.0),
        "act_scale": 0.05,
    }


def conv_layer_inputs(config: int, index: int, layer: ConvLayer, batch: int) -> Dict[str, object]:
    """Inputs of one layer of a CNN config: NCHW int8 activations ~ U{0..127} (post-ReLU), Gaussian-fit
    per-channel INT8 weights in OIHW, Bernoulli(0.5) rounding mask."""
    rng = rng_for(config, index)
    w, s = gaussian_weights_int8(rng, (layer.Cout, layer.Cin, layer.R, layer.S), layer.K)
    return {
        "X": uniform_int8(rng, (batch, layer.Cin, layer.H, layer.W), 0, 127),
        "W": w, "w_scale": s,
        "mask": bernoulli_mask(rng, w.shape),
        "act_scale": 0.02,
    }


def gemm_inputs(config: int, index: int, M: int, N: int, K: int, w_sigma=40.0, x_sigma=32.0) -> Dict[str, object]:
    """Config 4 style: W ~ clipped N(0, 40), X ~ clipped N(0, 32), per-channel scales U(1e-3, 1e-2)."""
    rng = rng_for(config, index)
    return {
        "W": clipped_normal_int8(rng, (N, K), w_sigma),
        "w_scale": channel_scales(rng, N),
        "mask": bernoulli_mask(rng, (N, K)),
        "X": clipped_normal_int8(rng, (M, K), x_sigma),
        "act_scale": 0.05,
    }


def vit_linear_inputs(index: int, M: int, K: int, N: int) -> Dict[str, object]:
    """Config 5 style: heavy-tailed Gaussian weights quantised per channel, X ~ clipped N(0, 32)."""
    rng = rng_for(5, index)
    w, s = heavy_tail_weights_int8(rng, (N, K))
    return {
        "W": w, "w_scale": s,
        "mask": bernoulli_mask(rng, (N, K)),
        "X": clipped_normal_int8(rng, (M, K), 32.0),
        "act_scale": 0.05,
    }


def oihw_to_ohwi_matrix(w_oihw: np.ndarray, ld: int = 0) -> np.ndarray:
    """Pure re-ordering: [Cout, Cin, R, S] -> [Cout, R*S*Cin] (optionally zero-padded to pitch ld)."""
    co = w_oihw.shape[0]
    m = np.ascontiguousarray(w_oihw.transpose(0, 2, 3, 1)).reshape(co, -1)
    if ld and ld > m.shape[1]:
        out = np.zeros((co, ld), dtype=m.dtype)
        out[:, : m.shape[1]] = m
        return out
    return m


# --------------------------------------------------------------------------- dependent chains (structure only)
def resnet_chain_plan(layers: List[ConvLayer]) -> List[Dict[str, object]]:
    """A ResNet-shaped layer table as ONE dependent chain: which tensor every layer reads and writes.  Pure
    structure (no arithmetic): stem -> 3x3 / 2 max pooling -> residual blocks (basic blocks c1, c2 or bottlenecks
    c1, c2, c3; the last convolution of a block adds the skip tensor -- the block's input, or its 1x1 down-sampling
    convolution `ds` -- before the ReLU) -> global average pooling -> classifier.  Steps:
      {"op": "conv", "layer": name, "src": tensor, "dst": tensor, "relu": bool, "skip": tensor or None}
      {"op": "maxpool", "src", "dst", "k", "stride", "pad"},  {"op": "avgpool", "src", "dst"},
      {"op": "fc", "layer": "fc", "src", "dst"}                      (fp32 logits, no requantisation)"""
    by = {L.name: L for L in layers}
    steps: List[Dict[str, object]] = [
        {"op": "conv", "layer": "conv1", "src": "input", "dst": "stem", "relu": True, "skip": None},
        {"op": "maxpool", "src": "stem", "dst": "pool", "k": 3, "stride": 2, "pad": 1},
    ]
    cur = "pool"
    for stage in range(1, 5):
        block = 0
        while f"l{stage}b{block}c1" in by:
            pre = f"l{stage}b{block}"
            convs = [c for c in ("c1", "c2", "c3") if pre + c in by]
            skip = cur
            if pre + "ds" in by:
                steps.append({"op": "conv", "layer": pre + "ds", "src": cur, "dst": pre + "ds", "relu": False, "skip": None})
                skip = pre + "ds"
            t = cur
            for c in convs[:-1]:
                steps.append({"op": "conv", "layer": pre + c, "src": t, "dst": pre + c, "relu": True, "skip": None})
                t = pre + c
            steps.append({"op": "conv", "layer": pre + convs[-1], "src": t, "dst": pre + "out", "relu": True, "skip": skip})
            cur = pre + "out"
            block += 1
    steps.append({"op": "avgpool", "src": cur, "dst": "pooled"})
    steps.append({"op": "fc", "layer": "fc", "src": "pooled", "dst": "logits"})
    return steps


def chain_weights(config: int, layers: List[ConvLayer]) -> Dict[str, Dict[str, np.ndarray]]:
    """Seeded weights of every layer of a chain: Gaussian fit + per-channel INT8 (OIHW), scales, rounding mask."""
    out = {}
    for i, L in enumerate(layers):
        rng = rng_for(config, 500 + i)
        w, s = gaussian_weights_int8(rng, (L.Cout, L.Cin, L.R, L.S), L.K)
        out[L.name] = {"W": w, "w_scale": s, "mask": bernoulli_mask(rng, w.shape)}
    return out
