"""Requantising epilogue (a layer's output as the next layer's INT8 activations): bit-exact against the oracle for the
GEMM in both modes and for the convolution, and a chained stack of layers that never leaves the device."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_padded(a):
    rows, cols = a.shape
    ld = -(-cols // 16) * 16
    buf = torch.zeros((rows, ld), dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    buf[:, :cols] = dev(a)
    return buf[:, :cols]


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (130, 200, 147), (300, 520, 1000), (1030, 1100, 640), (7, 24, 32)])
@pytest.mark.parametrize("relu,with_bias", [(True, False), (False, True)])
def test_gemm_both_modes(M, N, K, relu, with_bias):
    d = wl.gemm_inputs(95, M + N + K, M, N, K)
    W, X, mask, ws, sa = d["W"], d["X"], d["mask"], d["w_scale"], d["act_scale"]
    n, h = 8, 6
    rng = wl.rng_for(95, 7)
    bias = rng.normal(size=N).astype(np.float32) * 3 if with_bias else None
    out_scale = 0.37
    wh, wlo = oracle.decompose(W, mask, n, h, True)
    hi, lo = nq.nq_decompose(dev_padded(W), dev_padded(mask), n, h, True)
    Wd = dev_padded(W)
    Xd, wsd = dev_padded(X), dev(ws)
    bd = None if bias is None else dev(bias)
    got = nq.nq_gemm_full_q8(Xd, Wd, wsd, sa, out_scale, relu=relu, bias=bd).cpu().numpy()
    ref = oracle.requant(oracle.gemm_acc(X, W), ws, sa, 0, out_scale, bias=bias, relu=relu)
    assert np.array_equal(got, ref)
    got = nq.nq_gemm_part_q8(Xd, hi, N, n, h, wsd, sa, out_scale, relu=relu, bias=bd).cpu().numpy()
    ref = oracle.requant(oracle.gemm_acc(X, wh), ws, sa, n - h, out_scale, bias=bias, relu=relu)
    assert np.array_equal(got, ref)
    # nested full-bit mode: the full-bit result from the two packed parts
    got = nq.nq_gemm_nested_q8(Xd, hi, lo, N, n, h, wsd, sa, out_scale, relu=relu, bias=bd).cpu().numpy()
    ref = oracle.requant(oracle.gemm_acc(X, oracle.recompose(wh, wlo, n, h)), ws, sa, 0, out_scale, bias=bias, relu=relu)
    assert np.array_equal(got, ref)
    nq.nq_device_status()


C = wl.ConvLayer


@pytest.mark.parametrize("L", [C("c64", 64, 14, 14, 64, 3, 3, 1, 1), C("c128s2", 128, 13, 9, 72, 3, 3, 2, 1),
                               C("stem", 3, 32, 32, 64, 7, 7, 2, 3)], ids=lambda l: l.name)
def test_convolution_both_modes(L):
    batch, n, h = 3, 8, 6
    d = wl.conv_layer_inputs(96, sum(map(ord, L.name)), L, batch)
    X, W, mask, ws, sa = d["X"], d["W"], d["mask"], d["w_scale"], d["act_scale"]
    wh, _ = oracle.decompose(W, mask, n, h, True)
    ldw = -(-L.K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(W, ldw))[:, :L.K]
    m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ldw))[:, :L.K]
    hi, lo = nq.nq_decompose(w_mat, m_mat, n, h, True)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    out_scale = 0.9
    for part in (False, True):
        ref_acc = oracle.conv_acc(X, wh if part else W, L.stride, L.pad).transpose(0, 2, 3, 1)
        ref = oracle.requant(ref_acc, ws, sa, (n - h) if part else 0, out_scale, relu=True)
        got = nq.nq_conv_implicit_gemm_q8(dev(X), hi if part else w_mat, desc, dev(ws), sa, out_scale, relu=True,
                                          part_bit=part, n_bits=n, h_bits=h).cpu().numpy()
        assert np.array_equal(got, ref), (L.name, part)
    ref = oracle.requant(oracle.conv_acc(X, W, L.stride, L.pad).transpose(0, 2, 3, 1), ws, sa, 0, out_scale, relu=True)
    got = nq.nq_conv_implicit_gemm_nested_q8(dev(X), hi, lo, desc, dev(ws), sa, out_scale, relu=True, n_bits=n,
                                             h_bits=h).cpu().numpy()
    assert np.array_equal(got, ref), (L.name, "nested")
    nq.nq_device_status()


def test_three_chained_layers_stay_on_the_device():
    """conv 3x3 (64 -> 128, stride 2) -> conv 1x1 (128 -> 256) -> linear on the flattened map, each feeding the next
    its INT8 NHWC output; part-bit mode for the middle layer.  The oracle runs the same chain on the CPU."""
    batch = 2
    L1, L2 = C("a", 64, 12, 12, 128, 3, 3, 2, 1), C("b", 128, 6, 6, 256, 1, 1, 1, 0)
    d1, d2 = wl.conv_layer_inputs(97, 1, L1, batch), wl.conv_layer_inputs(97, 2, L2, batch)
    d3 = wl.gemm_inputs(97, 3, batch * 36, 64, 256)
    s1, s2, s3 = 0.02, 0.11, 0.23            # activation scales of the three layers' inputs
    # ---- oracle
    a1 = oracle.requant(oracle.conv_acc(d1["X"], d1["W"], 2, 1).transpose(0, 2, 3, 1), d1["w_scale"], s1, 0, s2)
    wh2, _ = oracle.decompose(d2["W"], d2["mask"], 8, 6, True)
    a2 = oracle.requant(oracle.conv_acc(a1.transpose(0, 3, 1, 2), wh2, 1, 0).transpose(0, 2, 3, 1), d2["w_scale"], s2, 2, s3)
    y_ref = oracle.dequant(oracle.gemm_acc(a2.reshape(-1, 256), d3["W"]), d3["w_scale"], s3, 0)
    # ---- device
    w1 = dev(wl.oihw_to_ohwi_matrix(d1["W"]))
    w2 = dev(wl.oihw_to_ohwi_matrix(d2["W"]))
    m2 = dev(wl.oihw_to_ohwi_matrix(d2["mask"]))
    hi2, _ = nq.nq_decompose(w2, m2, 8, 6, True)
    g1 = nq.nq_conv_implicit_gemm_q8(dev(d1["X"]), w1, nq.nq_conv_desc(batch, 64, 12, 12, 128, 3, 3, 2, 1, 1),
                                     dev(d1["w_scale"]), s1, s2)
    g2 = nq.nq_conv_implicit_gemm_q8(g1, hi2, nq.nq_conv_desc(batch, 128, 6, 6, 256, 1, 1, 1, 0, 0),
                                     dev(d2["w_scale"]), s2, s3, part_bit=True, n_bits=8, h_bits=6)
    _, y = nq.nq_gemm_full(g2.view(-1, 256), dev(d3["W"]), dev(d3["w_scale"]), s3)
    nq.nq_device_status()
    assert np.array_equal(g1.cpu().numpy(), a1) and np.array_equal(g2.cpu().numpy(), a2)
    assert np.array_equal(y.cpu().numpy(), y_ref)


def test_rejected_arguments():
    X = torch.zeros((16, 32), dtype=torch.int8, device="cuda")
    W = torch.zeros((16, 32), dtype=torch.int8, device="cuda")
    ws = torch.ones(16, device="cuda")
    with pytest.raises(nq.NqError):
        nq.nq_gemm_full_q8(X, W, ws, 1.0, 0.0)          # out_scale must be positive
