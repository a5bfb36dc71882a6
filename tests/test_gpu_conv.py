"""Parity of the implicit-GEMM convolution (full-bit and part-bit) with the CPU oracle's direct convolution.

The oracle works in the framework layout (NCHW activations, OIHW weights); the kernel's native layout is
NHWC activations and a [Cout, R*S*Cin] weight matrix, so the test re-orders (a pure permutation) on the way in
and out.  INT32 accumulators bit-exact, fp32 output equal to the oracle's (same rounding order).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def run_layer(L, batch, seed, n=8, h=6, nchw=True, check_y=True):
    d = wl.conv_layer_inputs(71, seed, L, batch)
    X, W, mask, ws, sa = d["X"], d["W"], d["mask"], d["w_scale"], d["act_scale"]
    if n < 8:                      # INTn nesting: INTn weights and n-bit activations in int8 containers
        W = (W >> (8 - n)).astype(np.int8)
        X = (X >> (8 - n)).astype(np.int8)
    wh, wlo = oracle.decompose(W, mask, n, h, True)
    K = L.K
    ldw = -(-K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(W, ldw))[:, :K]
    m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ldw))[:, :K]
    hi, lo = nq.nq_decompose(w_mat, m_mat, n, h, True)
    w_rec = torch.zeros((L.Cout, ldw), dtype=torch.int8, device="cuda")[:, :K]
    nq.nq_recompose(hi, lo, L.Cout, K, n, h, True, out=w_rec)
    assert torch.equal(w_rec, w_mat)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1 if nchw else 0)
    x_dev = dev(X if nchw else X.transpose(0, 2, 3, 1))
    wsd = dev(ws)
    for part in (False, True):
        ref = oracle.conv_acc(X, wh if part else W, L.stride, L.pad).transpose(0, 2, 3, 1)    # -> NHWC
        acc, y, _ = nq.nq_conv_implicit_gemm(x_dev, hi if part else w_rec, desc, wsd, sa, part_bit=part, n_bits=n,
                                             h_bits=h, want_acc=True)
        nq.nq_device_status()
        got = host(acc)
        assert got.shape == ref.shape
        assert np.array_equal(got, ref), (L, part, int(np.count_nonzero(got != ref)))
        if check_y:
            assert np.array_equal(host(y), oracle.dequant(ref, ws, sa, (n - h) if part else 0))
    if n in (6, 8) and h >= 2:
        # nested full-bit mode: the same full-bit result straight from the two packed parts
        ref = oracle.conv_acc(X, oracle.recompose(wh, wlo, n, h), L.stride, L.pad).transpose(0, 2, 3, 1)
        acc, y, _ = nq.nq_conv_implicit_gemm_nested(x_dev, hi, lo, desc, wsd, sa, n_bits=n, h_bits=h, want_acc=True)
        nq.nq_device_status()
        assert np.array_equal(host(acc), ref), (L, "nested")
        if check_y:
            assert np.array_equal(host(y), oracle.dequant(ref, ws, sa, 0))


C = wl.ConvLayer
SMALL = [
    # 64 input channels: two taps per stage, 64-byte swizzle; odd tap count leaves a half-filled last stage
    C("c64_3x3", 64, 14, 14, 64, 3, 3, 1, 1),
    C("c64_3x3_s2", 64, 14, 14, 128, 3, 3, 2, 1),
    C("c64_1x1_s2", 64, 14, 14, 128, 1, 1, 2, 0),
    C("c64_ragged", 64, 9, 11, 96, 3, 3, 1, 1),
    # multiples of 128 input channels: one tap and 128 channels per stage
    C("c128_3x3", 128, 14, 14, 128, 3, 3, 1, 1),
    C("c128_3x3_s2", 128, 14, 14, 256, 3, 3, 2, 1),
    C("c256_1x1", 256, 7, 7, 64, 1, 1, 1, 0),
    C("c256_1x1_s2", 256, 14, 14, 512, 1, 1, 2, 0),
    C("c128_7x7map", 128, 7, 7, 128, 3, 3, 1, 1),
    # anything else goes through the explicit patch matrix: the 3-channel stem, 16 and 32 channels
    C("stem", 3, 32, 32, 64, 7, 7, 2, 3),
    C("c16", 16, 10, 10, 32, 3, 3, 1, 1),
    C("c32_5x5", 32, 9, 9, 24, 5, 5, 1, 2),
]


@pytest.mark.parametrize("L", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("batch", [2, 3])
def test_small_layers_both_modes_both_layouts(L, batch):
    seed = sum(map(ord, L.name)) % 1000
    run_layer(L, batch, seed, nchw=True)
    run_layer(L, batch, seed + 1, nchw=False)


@pytest.mark.parametrize("h", [4, 5, 7])
def test_other_nestings(h):
    run_layer(C("c64", 64, 8, 8, 64, 3, 3, 1, 1), 4, 10 + h, h=h)
    run_layer(C("c128", 128, 8, 8, 64, 3, 3, 1, 1), 4, 20 + h, h=h)


@pytest.mark.parametrize("L", [C("c64_wide", 64, 40, 40, 64, 3, 3, 1, 1), C("c128_ragged", 128, 13, 9, 72, 3, 3, 2, 1)],
                         ids=lambda l: l.name)
def test_tile_stores_and_plain_stores_agree(L, debug_switch):
    """NHWC outputs go out as 4-D tile stores whose boxes follow the pixel rectangle of a tile (pixels outside the
    image are clipped by the store); the ordinary-store epilogue must give the same bytes."""
    run_layer(L, 3, 77)
    d = wl.conv_layer_inputs(71, 78, L, 3)
    ldw = -(-L.K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(d["W"], ldw))[:, :L.K]
    desc = nq.nq_conv_desc(3, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    x, ws = dev(d["X"]), dev(d["w_scale"])
    acc, y, _ = nq.nq_conv_implicit_gemm(x, w_mat, desc, ws, 0.02, want_acc=True, y_dtype=torch.bfloat16)
    debug_switch(nq.NQ_DEBUG_PLAIN_STORES)
    acc2, y2, _ = nq.nq_conv_implicit_gemm(x, w_mat, desc, ws, 0.02, want_acc=True, y_dtype=torch.bfloat16)
    nq.nq_device_status()
    assert torch.equal(acc, acc2) and torch.equal(y.view(torch.int16), y2.view(torch.int16))


@pytest.mark.parametrize("n,h", [(6, 3), (6, 4), (6, 5), (8, 3)])
def test_int6_nesting_and_three_bit_high_part(n, h):
    """INT6 nesting (6-bit weights and activations, h in {3, 4, 5}) and the 3-bit high part of INT8 nesting through
    both convolution modes, both operating modes."""
    run_layer(C("c64", 64, 10, 10, 64, 3, 3, 1, 1), 3, 30 + n + h, n=n, h=h)
    run_layer(C("c128", 128, 9, 9, 96, 3, 3, 2, 1), 3, 40 + n + h, n=n, h=h)
    run_layer(C("stem", 3, 20, 20, 32, 7, 7, 2, 3), 2, 50 + n + h, n=n, h=h)


def test_pointwise_convolution_equals_the_gemm_entry_point():
    L = C("pw", 128, 6, 6, 96, 1, 1, 1, 0)
    d = wl.conv_layer_inputs(72, 0, L, 5)
    x_nhwc = dev(d["X"].transpose(0, 2, 3, 1))
    w = dev(d["W"].reshape(96, 128))
    ws = dev(d["w_scale"])
    desc = nq.nq_conv_desc(5, 128, 6, 6, 96, 1, 1, 1, 0, 0)
    acc_c, y_c, _ = nq.nq_conv_implicit_gemm(x_nhwc, w, desc, ws, 0.02, want_acc=True)
    acc_g, y_g = nq.nq_gemm_full(x_nhwc.view(-1, 128), w, ws, 0.02, want_acc=True)
    assert torch.equal(acc_c.view(-1, 96), acc_g) and torch.equal(y_c.view(-1, 96), y_g)


@pytest.mark.parametrize("name", ["l1b0c1", "l2b0c1", "l2b0ds", "l3b0c2", "l4b0c2", "conv1", "fc"])
def test_resnet18_layers_at_benchmark_size_sampled_pixels(name):
    """Config-2 layers at batch 32 in the launch configuration the benchmark times; the oracle evaluates
    the convolution at sampled output pixels (corners, tile borders, random), all channels."""
    L = next(l for l in wl.resnet18_layers() if l.name == name)
    batch = 32
    d = wl.conv_layer_inputs(2, 5, L, batch)
    X, W, mask, ws, sa = d["X"], d["W"], d["mask"], d["w_scale"], d["act_scale"]
    wh, _ = oracle.decompose(W, mask, 8, 6, True)
    K = L.K
    ldw = -(-K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(W, ldw))[:, :K]
    m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ldw))[:, :K]
    hi, lo = nq.nq_decompose(w_mat, m_mat, 8, 6, True)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    rng = wl.rng_for(2, 77)
    Ho, Wo = L.Ho, L.Wo
    fixed = [(0, 0, 0), (0, 0, Wo - 1), (0, Ho - 1, 0), (batch - 1, Ho - 1, Wo - 1), (1, min(7, Ho - 1), min(8, Wo - 1)),
             (batch - 1, 0, 0), (15, Ho // 2, Wo // 2)]
    rand = [(int(rng.integers(batch)), int(rng.integers(Ho)), int(rng.integers(Wo))) for _ in range(40)]
    pix = np.array(sorted(set(fixed + rand)), dtype=np.int64)
    x_dev, wsd = dev(X), dev(ws)
    for part in (False, True):
        acc, y, _ = nq.nq_conv_implicit_gemm(x_dev, hi if part else w_mat, desc, wsd, sa, part_bit=part, n_bits=8, h_bits=6,
                                             want_acc=True)
        nq.nq_device_status()
        ref = oracle.conv_acc_pixels(X, wh if part else W, L.stride, L.pad, pix)
        idx = torch.from_numpy(pix).cuda()
        got = host(acc[idx[:, 0], idx[:, 1], idx[:, 2]])
        assert np.array_equal(got, ref), (name, part)
        got_y = host(y[idx[:, 0], idx[:, 1], idx[:, 2]])
        assert np.array_equal(got_y, oracle.dequant(ref, ws, sa, 2 if part else 0))
        # whole-output checksum: sum over channels of acc = x-patch . (sum over channels of w), at the sampled pixels
        # is covered above; over the whole tensor, the channel sums of the accumulator must match an int64 einsum
        if L.R == 1 and L.stride == 1:
            xs = X.astype(np.int64).sum(axis=(0, 2, 3))                         # [Cin]
            wref = (wh if part else W).astype(np.int64).reshape(L.Cout, L.Cin)
            assert np.array_equal(host(acc).astype(np.int64).sum(axis=(0, 1, 2)), wref @ xs)


def test_rejected_arguments():
    desc = nq.nq_conv_desc(1, 64, 8, 8, 64, 3, 3, 1, 1, 1)
    x = torch.zeros((1, 64, 8, 8), dtype=torch.int8, device="cuda")
    w = torch.zeros((64, 576), dtype=torch.int8, device="cuda")
    ws = torch.ones(64, device="cuda")
    assert nq.nq_conv_workspace_bytes(desc) == 64 * 64
    small = torch.zeros(2048, dtype=torch.uint8, device="cuda")
    with pytest.raises(nq.NqError) as e:
        nq.nq_conv_implicit_gemm(x, w, desc, ws, 1.0, workspace=small)
    assert e.value.status == 4
    bad = nq.nq_conv_desc(1, 64, 2, 2, 64, 5, 5, 1, 0, 0)
    assert nq.nq_conv_workspace_bytes(bad) == -1
