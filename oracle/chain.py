"""A ResNet-shaped model as one dependent chain, composed from the oracle's own functions.

TEST INFRASTRUCTURE ONLY (like the rest of ``oracle/``).  The paper runs its models with 8-bit activations and
nested weights but defines neither the hand-over between layers nor the blocks' arithmetic; the chain below is the
library's own definition (parity unpinned by the paper), built from steps that are each pinned on their own:
convolution accumulators (``conv_acc``), the requantising hand-over with or without a skip tensor (``requant``,
``requant_res``), pooling (``maxpool_nhwc``, ``avgpool_requant_nhwc``) and the classifier's dequantisation.

Activation scales: when none are given, every tensor's scale is chosen from the data as max|v| / 127 of its
pre-rounding values (a calibration pass); the scales found are returned so that another implementation can be run
with exactly the same numbers.
"""
from __future__ import annotations

import numpy as np

from . import (avgpool_requant_nhwc, conv_acc, decompose, dequant, gemm_acc, maxpool_nhwc, requant, requant_res)


def _nchw(x_nhwc):
    return np.ascontiguousarray(x_nhwc.transpose(0, 3, 1, 2))


def _nhwc(x_nchw):
    return np.ascontiguousarray(x_nchw.transpose(0, 2, 3, 1))


def run_resnet_chain(plan, layers, weights, x_nchw, in_scale, part_bit=False, n_bits=8, h_bits=6, scales=None):
    """Runs the chain of workloads.resnet_chain_plan.  weights[name] = {"W": int8 OIHW, "w_scale", "mask"}.
    part_bit: every layer uses w_high alone with the inflated scale (Eq. 9); otherwise the INTn weights (Eq. 2).
    Returns (tensors: name -> int8 NHWC array (logits: fp32 [B, classes]), scales: name -> float)."""
    by = {L.name: L for L in layers}
    l_shift = (n_bits - h_bits) if part_bit else 0
    calibrate = scales is None
    scales = {} if calibrate else dict(scales)
    scales["input"] = float(in_scale)
    t = {"input": _nhwc(np.asarray(x_nchw, dtype=np.int8))}

    def weight_of(name):
        w = weights[name]
        if part_bit:
            wh, _ = decompose(w["W"], w["mask"], n_bits, h_bits, True)
            return wh
        return w["W"]

    for st in plan:
        op = st["op"]
        if op == "conv":
            L = by[st["layer"]]
            w = weights[st["layer"]]
            acc = _nhwc(conv_acc(_nchw(t[st["src"]]), weight_of(st["layer"]), L.stride, L.pad))     # [B, Ho, Wo, Cout]
            skip = st["skip"]
            if calibrate:
                v = dequant(acc, w["w_scale"], scales[st["src"]], l_shift).astype(np.float64)
                if skip is not None:
                    v = v + t[skip].astype(np.float64) * scales[skip]
                if st["relu"]:
                    v = np.maximum(v, 0.0)
                scales[st["dst"]] = float(np.float32(max(float(np.max(np.abs(v))), 1e-6) / 127.0))
            if skip is None:
                q = requant(acc, w["w_scale"], scales[st["src"]], l_shift, scales[st["dst"]], relu=st["relu"])
            else:
                q = requant_res(acc, w["w_scale"], scales[st["src"]], l_shift, scales[st["dst"]], t[skip], scales[skip],
                                relu=st["relu"])
            t[st["dst"]] = q
        elif op == "maxpool":
            t[st["dst"]] = maxpool_nhwc(t[st["src"]], st["k"], st["stride"], st["pad"])
            scales[st["dst"]] = scales[st["src"]]
        elif op == "avgpool":
            x = t[st["src"]]
            if calibrate:
                mean = x.astype(np.float64).mean(axis=(1, 2)) * scales[st["src"]]
                scales[st["dst"]] = float(np.float32(max(float(np.max(np.abs(mean))), 1e-6) / 127.0))
            t[st["dst"]] = avgpool_requant_nhwc(x, scales[st["src"]], scales[st["dst"]])
        elif op == "fc":
            w = weights[st["layer"]]
            wm = weight_of(st["layer"]).reshape(w["W"].shape[0], -1)
            acc = gemm_acc(t[st["src"]], wm)
            t[st["dst"]] = dequant(acc, w["w_scale"], scales[st["src"]], l_shift)
        else:
            raise ValueError(op)
    return t, scales
