"""A ResNet-shaped model run as ONE dependent chain on the device: every layer's INT8 output is the next layer's
input.  This module only strings library calls together (argument marshalling and buffer book-keeping); every step
of the arithmetic runs in the kernels behind ``include/nq.h``:

  convolution + requantising epilogue (ReLU, skip tensor of a residual block)   nq_conv_implicit_gemm_q8[_res]
  the same in nested full-bit mode (weights rebuilt from the two packed parts)    nq_conv_implicit_gemm_nested_q8[_res]
  stem max pooling, global average pooling                                        nq_maxpool_nhwc_i8, nq_avgpool_requant_nhwc_i8
  classifier (fp32 logits)                                                        nq_gemm_full / nq_gemm_part / nq_gemm_nested

Modes: "full" (INT8 weights resident, Eq. 2), "part" (packed w_high alone, scale inflated by 2^l, Eq. 9), "nested"
(full-bit results straight from packed w_high and compensated w_low, Eq. 5 inside the kernel).
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as nq
from .workloads import ConvLayer


class ResNetChain:
    def __init__(self, layers: List[ConvLayer], plan: List[dict], weights: Dict[str, dict], batch: int, in_scale: float,
                 n_bits: int = 8, h_bits: int = 6, device="cuda", input_nchw: bool = True):
        self.layers = {L.name: L for L in layers}
        self.plan, self.batch, self.n, self.h = plan, batch, n_bits, h_bits
        self.dev = torch.device(device)
        self.input_nchw = input_nchw
        self.scales: Dict[str, float] = {"input": float(in_scale)}
        self.w: Dict[str, dict] = {}
        work = 0
        for st in plan:
            if st["op"] not in ("conv", "fc"):
                continue
            L = self.layers[st["layer"]]
            hw = weights[L.name]
            ldw = -(-L.K // 16) * 16
            ohwi = np.ascontiguousarray(hw["W"].transpose(0, 2, 3, 1)).reshape(L.Cout, L.K)
            mask = np.ascontiguousarray(hw["mask"].transpose(0, 2, 3, 1)).reshape(L.Cout, L.K)
            w_mat = torch.zeros((L.Cout, ldw), dtype=torch.int8, device=self.dev)
            m_mat = torch.zeros((L.Cout, ldw), dtype=torch.uint8, device=self.dev)
            w_mat[:, :L.K] = torch.from_numpy(ohwi).to(self.dev)
            m_mat[:, :L.K] = torch.from_numpy(mask).to(self.dev)
            hi, lo = nq.nq_decompose(w_mat[:, :L.K], m_mat[:, :L.K], n_bits, h_bits, True)
            nchw = 1 if (st["op"] == "conv" and st["src"] == "input" and input_nchw) else 0
            desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, nchw)
            work = max(work, nq.nq_conv_workspace_bytes(desc))
            self.w[L.name] = {"w": w_mat[:, :L.K], "hi": hi, "lo": lo, "desc": desc,
                              "ws": torch.from_numpy(np.ascontiguousarray(hw["w_scale"])).to(self.dev)}
        self.work = torch.empty(work + 2048, dtype=torch.uint8, device=self.dev)
        # one buffer per tensor of the chain (a skip tensor must outlive the layers between its two uses)
        self.t: Dict[str, torch.Tensor] = {}
        for st in plan:
            if st["op"] == "conv":
                L = self.layers[st["layer"]]
                self.t[st["dst"]] = torch.empty((batch, L.Ho, L.Wo, L.Cout), dtype=torch.int8, device=self.dev)
            elif st["op"] == "maxpool":
                b, h, w, c = self.t[st["src"]].shape
                ho = (h + 2 * st["pad"] - st["k"]) // st["stride"] + 1
                wo = (w + 2 * st["pad"] - st["k"]) // st["stride"] + 1
                self.t[st["dst"]] = torch.empty((b, ho, wo, c), dtype=torch.int8, device=self.dev)
            elif st["op"] == "avgpool":
                self.t[st["dst"]] = torch.empty((batch, self.t[st["src"]].shape[3]), dtype=torch.int8, device=self.dev)
            elif st["op"] == "fc":
                self.t[st["dst"]] = torch.empty((batch, self.layers[st["layer"]].Cout), dtype=torch.float32, device=self.dev)

    # ------------------------------------------------------------------ scales
    def set_scales(self, scales: Dict[str, float]) -> None:
        self.scales.update({k: float(v) for k, v in scales.items()})

    def calibrate(self, x: torch.Tensor, mode: str = "full") -> Dict[str, float]:
        """Chooses every tensor's activation scale from the data (max |pre-rounding value| / 127), layer by layer:
        the fp32-output convolution gives the values, torch reduces them.  Set-up only, not part of a timed run."""
        l = (self.n - self.h) if mode == "part" else 0
        self.t["input"] = x
        for st in self.plan:
            if st["op"] == "conv":
                e = self.w[st["layer"]]
                _, v, _ = nq.nq_conv_implicit_gemm(self.t[st["src"]], e["hi"] if mode == "part" else e["w"], e["desc"], e["ws"],
                                                   self.scales[st["src"]], part_bit=(mode == "part"), n_bits=self.n,
                                                   h_bits=self.h, workspace=self.work)
                if st["skip"] is not None:
                    v = v + self.t[st["skip"]].float() * self.scales[st["skip"]]
                if st["relu"]:
                    v = torch.relu(v)
                self.scales[st["dst"]] = float(np.float32(max(float(v.abs().max()), 1e-6) / 127.0))
                del v
                self._step(st, mode)
            elif st["op"] == "avgpool":
                mean = self.t[st["src"]].float().mean(dim=(1, 2)) * self.scales[st["src"]]
                self.scales[st["dst"]] = float(np.float32(max(float(mean.abs().max()), 1e-6) / 127.0))
                self._step(st, mode)
            else:
                if st["op"] == "maxpool":
                    self.scales[st["dst"]] = self.scales[st["src"]]
                self._step(st, mode)
        _ = l
        return dict(self.scales)

    # ------------------------------------------------------------------ one pass
    def _step(self, st: dict, mode: str) -> None:
        op = st["op"]
        if op == "conv":
            e = self.w[st["layer"]]
            src, dst = self.t[st["src"]], self.t[st["dst"]]
            s_in, s_out = self.scales[st["src"]], self.scales[st["dst"]]
            skip = st["skip"]
            if mode == "nested":
                if skip is None:
                    nq.nq_conv_implicit_gemm_nested_q8(src, e["hi"], e["lo"], e["desc"], e["ws"], s_in, s_out, relu=st["relu"],
                                                       n_bits=self.n, h_bits=self.h, workspace=self.work, y_out=dst)
                else:
                    nq.nq_conv_implicit_gemm_nested_q8_res(src, e["hi"], e["lo"], e["desc"], e["ws"], s_in, self.t[skip],
                                                           self.scales[skip], s_out, relu=st["relu"], n_bits=self.n,
                                                           h_bits=self.h, workspace=self.work, y_out=dst)
            else:
                part = mode == "part"
                wt = e["hi"] if part else e["w"]
                if skip is None:
                    nq.nq_conv_implicit_gemm_q8(src, wt, e["desc"], e["ws"], s_in, s_out, relu=st["relu"], part_bit=part,
                                                n_bits=self.n, h_bits=self.h, workspace=self.work, y_out=dst)
                else:
                    nq.nq_conv_implicit_gemm_q8_res(src, wt, e["desc"], e["ws"], s_in, self.t[skip], self.scales[skip], s_out,
                                                    relu=st["relu"], part_bit=part, n_bits=self.n, h_bits=self.h,
                                                    workspace=self.work, y_out=dst)
        elif op == "maxpool":
            nq.nq_maxpool_nhwc_i8(self.t[st["src"]], st["k"], st["stride"], st["pad"], y_out=self.t[st["dst"]])
        elif op == "avgpool":
            nq.nq_avgpool_requant_nhwc_i8(self.t[st["src"]], self.scales[st["src"]], self.scales[st["dst"]],
                                          y_out=self.t[st["dst"]])
        elif op == "fc":
            e = self.w[st["layer"]]
            x, y = self.t[st["src"]], self.t[st["dst"]]
            s_in = self.scales[st["src"]]
            if mode == "full":
                nq.nq_gemm_full(x, e["w"], e["ws"], s_in, y_out=y)
            elif mode == "part":
                nq.nq_gemm_part(x, e["hi"], e["w"].shape[0], self.n, self.h, e["ws"], s_in, y_out=y)
            else:
                nq.nq_gemm_nested(x, e["hi"], e["lo"], e["w"].shape[0], self.n, self.h, e["ws"], s_in, y_out=y)
        else:
            raise ValueError(op)

    def run(self, x: torch.Tensor, mode: str = "full") -> torch.Tensor:
        """One pass of the chain on the current stream; x is int8 NCHW (or NHWC when input_nchw is False).
        Returns the logits tensor (fp32 [batch, classes]); every intermediate stays in self.t."""
        self.t["input"] = x
        for st in self.plan:
            self._step(st, mode)
        return self.t["logits"]

    def kernels_per_pass(self) -> int:
        """Kernel launches of one pass (a layout pre-pass counts: the stem's patch matrix)."""
        n = 0
        for st in self.plan:
            n += 1
            if st["op"] == "conv" and nq.nq_conv_workspace_bytes(self.w[st["layer"]]["desc"]) > 0:
                n += 1
        return n
