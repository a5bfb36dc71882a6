"""Chained inference on the device against the oracle's chain: the residual hand-over, the pooling kernels, and
whole ResNet-shaped models run as ONE dependent chain (stem -> pooling -> residual blocks -> pooling -> classifier)
in full-bit, part-bit and nested full-bit mode.  Everything is integer or rounds identically on both sides, so every
intermediate INT8 tensor is compared bit for bit and the fp32 logits for equality."""
import numpy as np
import pytest
import torch

import oracle
from oracle import chain as ochain
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl
from paper_2506_17870_b200.chain import ResNetChain

pytestmark = pytest.mark.gpu
C = wl.ConvLayer


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


LAYERS = [C("c64", 64, 14, 14, 64, 3, 3, 1, 1), C("c128", 128, 9, 11, 256, 1, 1, 1, 0), C("c128s2", 128, 13, 9, 80, 3, 3, 2, 1),
          C("stem", 3, 20, 20, 32, 7, 7, 2, 3), C("ragged_n", 64, 8, 8, 72, 3, 3, 1, 1), C("odd_n", 64, 6, 6, 19, 1, 1, 1, 0)]


@pytest.mark.parametrize("L", LAYERS, ids=lambda l: l.name)
@pytest.mark.parametrize("relu", [True, False])
def test_requantising_convolution_with_a_skip_tensor(L, relu):
    batch, n, h = 3, 8, 6
    d = wl.conv_layer_inputs(72, len(L.name) + L.Cout, L, batch)
    rng = wl.rng_for(72, 900 + L.Cout)
    res = wl.uniform_int8(rng, (batch, L.Ho, L.Wo, L.Cout))
    bias = rng.normal(size=L.Cout).astype(np.float32)
    res_scale, out_scale = 0.037, 0.41
    X, W, mask, ws, sa = d["X"], d["W"], d["mask"], d["w_scale"], d["act_scale"]
    wh, wlo = oracle.decompose(W, mask, n, h, True)
    ldw = -(-L.K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(W, ldw))[:, :L.K]
    m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ldw))[:, :L.K]
    hi, lo = nq.nq_decompose(w_mat, m_mat, n, h, True)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    x_dev, wsd, res_d, bias_d = dev(X), dev(ws), dev(res), dev(bias)
    for mode in ("full", "part", "nested"):
        Wref, l = (wh, n - h) if mode == "part" else (W, 0)
        acc = np.ascontiguousarray(oracle.conv_acc(X, Wref, L.stride, L.pad).transpose(0, 2, 3, 1))
        ref = oracle.requant_res(acc, ws, sa, l, out_scale, res, res_scale, bias=bias, relu=relu)
        if mode == "nested":
            got = nq.nq_conv_implicit_gemm_nested_q8_res(x_dev, hi, lo, desc, wsd, sa, res_d, res_scale, out_scale, relu=relu,
                                                         n_bits=n, h_bits=h, bias=bias_d)
        else:
            got = nq.nq_conv_implicit_gemm_q8_res(x_dev, hi if mode == "part" else w_mat, desc, wsd, sa, res_d, res_scale,
                                                  out_scale, relu=relu, part_bit=(mode == "part"), n_bits=n, h_bits=h, bias=bias_d)
        nq.nq_device_status()
        assert np.array_equal(host(got), ref), mode


@pytest.mark.parametrize("shape,k,stride,pad", [((2, 112, 112, 64), 3, 2, 1), ((3, 9, 11, 5), 3, 2, 1), ((1, 7, 7, 48), 2, 2, 0),
                                                ((2, 5, 5, 16), 3, 1, 1)])
def test_max_pooling(shape, k, stride, pad):
    rng = wl.rng_for(73, shape[1] + shape[3])
    x = wl.uniform_int8(rng, shape)
    assert np.array_equal(host(nq.nq_maxpool_nhwc_i8(dev(x), k, stride, pad)), oracle.maxpool_nhwc(x, k, stride, pad))


@pytest.mark.parametrize("shape", [(4, 7, 7, 512), (3, 5, 3, 19), (2, 14, 14, 2048)])
def test_global_average_pooling(shape):
    rng = wl.rng_for(74, shape[3])
    x = wl.uniform_int8(rng, shape, 0, 127)
    for s_in, s_out in ((0.05, 0.03), (2.69, 1.58)):
        assert np.array_equal(host(nq.nq_avgpool_requant_nhwc_i8(dev(x), s_in, s_out)), oracle.avgpool_requant_nhwc(x, s_in, s_out))


def run_model_chain(layers, batch, config):
    plan = wl.resnet_chain_plan(layers)
    weights = wl.chain_weights(config, layers)
    x = wl.uniform_int8(wl.rng_for(config, 999), (batch, 3, 224, 224), 0, 127)
    gpu = ResNetChain(layers, plan, weights, batch, 0.02)
    x_dev = dev(x)
    ref_full = None
    for mode in ("full", "part", "nested"):
        if mode == "nested":
            ref, scales = ref_full                          # nested full-bit computes exactly the full-bit model
        else:
            ref, scales = ochain.run_resnet_chain(plan, layers, weights, x, 0.02, part_bit=(mode == "part"))
            if mode == "full":
                ref_full = (ref, scales)
        gpu.set_scales(scales)
        logits = gpu.run(x_dev, mode)
        nq.nq_device_status()
        for st in plan:
            name = st["dst"]
            if name == "logits":
                continue
            assert np.array_equal(host(gpu.t[name]), ref[name]), (mode, name)
        assert np.array_equal(host(logits), ref["logits"]), mode
    # the chain is non-trivial: activations neither vanish nor saturate everywhere
    last = ref_full[0]["pooled"]
    assert 0.2 < float((last != 0).mean()) and float((np.abs(last.astype(np.int32)) == 127).mean()) < 0.2


def test_resnet18_shaped_model_as_one_dependent_chain():
    run_model_chain(wl.resnet18_layers(), 2, 2)


def test_resnet101_shaped_model_as_one_dependent_chain():
    run_model_chain(wl.resnet101_layers(), 1, 3)


def test_device_calibration_gives_usable_scales_and_a_stable_chain():
    layers = wl.resnet18_layers()
    plan = wl.resnet_chain_plan(layers)
    gpu = ResNetChain(layers, plan, wl.chain_weights(2, layers), 2, 0.02)
    x = dev(wl.uniform_int8(wl.rng_for(2, 998), (2, 3, 224, 224), 0, 127))
    scales = gpu.calibrate(x, "full")
    assert all(np.isfinite(v) and v > 0 for v in scales.values())
    a = gpu.run(x, "full").clone()
    b = gpu.run(x, "nested").clone()
    nq.nq_device_status()
    assert torch.equal(a, b) and float(a.abs().max()) > 0
