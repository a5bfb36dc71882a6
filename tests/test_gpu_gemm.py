"""Parity of the nested INT8 GEMM (full-bit and part-bit) with the CPU oracle.

INT32 accumulators: bit-exact.  Dequantised output: the stated bar is max-abs error <= 1e-5 of the
largest output magnitude; both sides round in the same order, so the test also reports (and for
fp32 requires) exact equality.  bf16 output: equal to the round-to-nearest-even bf16 of the
oracle's fp32 value.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_padded(a, multiple=16):
    """Device copy whose row pitch is a multiple of 16 bytes (TMA's stride rule); returns the view."""
    rows, cols = a.shape
    ld = -(-cols // multiple) * multiple
    buf = torch.zeros((rows, ld), dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    buf[:, :cols] = dev(a)
    return buf[:, :cols]


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def check_outputs(acc_gpu, y_gpu, acc_ref, w_scale, act_scale, l_shift, bias=None, bf16=False):
    assert np.array_equal(host(acc_gpu), acc_ref), "int32 accumulators differ"
    y_ref, y64 = oracle.dequant(acc_ref, w_scale, act_scale, l_shift, bias=bias, want_ref=True)
    if bf16:
        got = host(y_gpu.view(torch.int16)).view(np.uint16)
        assert np.array_equal(got, oracle.f32_to_bf16_bits(y_ref))
    else:
        got = host(y_gpu)
        err = np.max(np.abs(got.astype(np.float64) - y_ref.astype(np.float64)))
        assert err <= REL_TOL * np.max(np.abs(y_ref)), err
        assert np.array_equal(got, y_ref)
        assert np.max(np.abs(got - y64)) <= 1e-6 * np.max(np.abs(y64)) + 1e-30


def run_both_modes(d, n, h, bias=None, bf16=False):
    W, X, mask, ws, sa = d["W"], d["X"], d["mask"], d["w_scale"], d["act_scale"]
    N, K = W.shape
    l = n - h
    wh, wlo = oracle.decompose(W, mask, n, h, True)
    Xd, wsd = dev_padded(X), dev(ws)
    bd = None if bias is None else dev(bias)
    ydt = torch.bfloat16 if bf16 else torch.float32
    hi, lo = nq.nq_decompose(dev_padded(W), dev_padded(mask), n, h, True)
    # full-bit: on the weights the GPU recomposed itself
    Wfull = torch.zeros((N, -(-K // 16) * 16), dtype=torch.int8, device="cuda")[:, :K]
    nq.nq_recompose(hi, lo, N, K, n, h, True, out=Wfull)
    acc, y = nq.nq_gemm_full(Xd, Wfull, wsd, sa, bias=bd, want_acc=True, y_dtype=ydt)
    check_outputs(acc, y, oracle.gemm_acc(X, oracle.recompose(wh, wlo, n, h)), ws, sa, 0, bias, bf16)
    # part-bit: on the packed high part
    acc_p, y_p = nq.nq_gemm_part(Xd, hi, N, n, h, wsd, sa, bias=bd, want_acc=True, y_dtype=ydt)
    check_outputs(acc_p, y_p, oracle.gemm_acc(X, wh), ws, sa, l, bias, bf16)
    nq.nq_device_status()


def test_config1_single_linear_layer_int8_nesting_int6():
    c = wl.config1()
    run_both_modes(c, 8, 6)
    run_both_modes(c, 8, 6, bf16=True)


# several tiles in every direction, ragged M / N / K tails, every N-tile width, one row, K not a multiple of 16
SHAPES = [(64, 256, 256), (130, 200, 147), (300, 520, 1000), (128, 64, 128), (1, 1000, 512),
          (257, 96, 4099), (515, 300, 130), (7, 24, 32)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_ragged_shapes_both_modes(M, N, K):
    d = wl.gemm_inputs(81, M + N + K, M, N, K)
    run_both_modes(d, 8, 6)


@pytest.mark.parametrize("h", [1, 2, 3, 4, 5, 6, 7])
def test_every_part_bit_width(h):
    d = wl.gemm_inputs(82, h, 200, 384, 640)
    run_both_modes(d, 8, h)


def test_int6_nesting_and_bias_and_bf16():
    rng = wl.rng_for(83)
    d = wl.gemm_inputs(83, 1, 160, 272, 384)
    d["W"] = wl.uniform_int8(rng, (272, 384), -32, 31)
    d["X"] = wl.uniform_int8(rng, (160, 384), -32, 31)
    bias = rng.normal(size=272).astype(np.float32)
    run_both_modes(d, 6, 4, bias=bias)
    run_both_modes(d, 6, 5, bias=bias, bf16=True)
    d8 = wl.gemm_inputs(83, 2, 96, 520, 256)
    run_both_modes(d8, 8, 4, bias=rng.normal(size=520).astype(np.float32), bf16=True)


def test_extreme_values_fill_the_accumulator_range():
    K = 16384
    X = np.full((128, K), -128, dtype=np.int8)
    W = np.full((64, K), -128, dtype=np.int8)
    ws = np.full(64, 0.01, dtype=np.float32)
    acc, y = nq.nq_gemm_full(dev(X), dev(W), dev(ws), 0.05, want_acc=True)
    assert torch.all(acc == K * 128 * 128)
    W[:] = 127
    acc, _ = nq.nq_gemm_full(dev(X), dev(W), dev(ws), 0.05, want_acc=True)
    assert torch.all(acc == -K * 128 * 127)


def test_full_equals_shifted_part_plus_low_contribution():
    # Eq. 5 under the contraction, all three terms from the GPU: X W^T = 2^l X Wh^T + X Wl^T
    d = wl.gemm_inputs(84, 0, 256, 512, 1024)
    n, h = 8, 5
    hi, lo = nq.nq_decompose(dev(d["W"]), dev(d["mask"]), n, h, True)
    X, ws = dev(d["X"]), dev(d["w_scale"])
    full, _ = nq.nq_gemm_full(X, nq.nq_recompose(hi, lo, 512, 1024, n, h, True), ws, 0.05, want_acc=True, y_dtype=None)
    part, _ = nq.nq_gemm_part(X, hi, 512, n, h, ws, 0.05, want_acc=True, y_dtype=None)
    low, _ = nq.nq_gemm_full(X, nq.nq_unpack(lo, 4, 512, 1024), ws, 0.05, want_acc=True, y_dtype=None)
    assert torch.equal(full.long(), (part.long() << 3) + low.long())


@pytest.mark.parametrize("h", [1, 2, 3, 4, 5, 6, 7])
def test_wide_ragged_gemm_narrow_fields(h, debug_switch):
    """Large enough for the CTA-pair kernel, whose unpack warps read fields of 1, 2 and 4 bits straight from the
    packed matrix: ragged in M, N and K, every width checked against the oracle, and bit for bit against the same
    launch with every width fed through the shared-memory ring of packed tiles."""
    M, N, K = 3500, 1100, 1100
    d = wl.gemm_inputs(89, h, M, N, K)
    wh, _ = oracle.decompose(d["W"], d["mask"], 8, h, True)
    hi, _ = nq.nq_decompose(dev_padded(d["W"]), dev_padded(d["mask"]), 8, h, True)
    Xd, wsd = dev_padded(d["X"]), dev(d["w_scale"])
    acc, y = nq.nq_gemm_part(Xd, hi, N, 8, h, wsd, d["act_scale"], want_acc=True)
    nq.nq_device_status()
    check_outputs(acc, y, oracle.gemm_acc(d["X"], wh), d["w_scale"], d["act_scale"], 8 - h)
    debug_switch(nq.NQ_DEBUG_PACKED_RING)
    acc2, y2 = nq.nq_gemm_part(Xd, hi, N, 8, h, wsd, d["act_scale"], want_acc=True)
    nq.nq_device_status()
    assert torch.equal(acc, acc2) and torch.equal(y, y2)


@pytest.mark.parametrize("M,N,K,bf16", [(300, 520, 1000, False), (300, 520, 1000, True), (1030, 1100, 640, True),
                                         (130, 40, 147, False), (2100, 72, 256, True)])
def test_tile_stores_and_plain_stores_agree(M, N, K, bf16, debug_switch):
    """The epilogue writes aligned outputs with TMA tile stores (ragged rows and columns clipped by the store) and
    everything else with ordinary stores: both against the oracle, and bit for bit against each other."""
    d = wl.gemm_inputs(90, M + N + K, M, N, K)
    run_both_modes(d, 8, 6, bf16=bf16)
    hi, _ = nq.nq_decompose(dev_padded(d["W"]), dev_padded(d["mask"]), 8, 6, True)
    Xd, wsd = dev_padded(d["X"]), dev(d["w_scale"])
    ydt = torch.bfloat16 if bf16 else torch.float32
    acc, y = nq.nq_gemm_part(Xd, hi, N, 8, 6, wsd, d["act_scale"], want_acc=True, y_dtype=ydt)
    debug_switch(nq.NQ_DEBUG_PLAIN_STORES)
    acc2, y2 = nq.nq_gemm_part(Xd, hi, N, 8, 6, wsd, d["act_scale"], want_acc=True, y_dtype=ydt)
    nq.nq_device_status()
    assert torch.equal(acc, acc2) and torch.equal(y.view(torch.int16 if bf16 else torch.int32),
                                                  y2.view(torch.int16 if bf16 else torch.int32))


@pytest.mark.parametrize("M,N,K", [(200, 8, 64), (33, 16, 128), (129, 4, 32)])
def test_outputs_narrower_than_a_store_box(M, N, K):
    """Output rows shorter than the 64-byte box of a tile store (aligned pitch, so the tile-store path is taken)."""
    d = wl.gemm_inputs(91, M + N + K, M, N, K)
    run_both_modes(d, 8, 6)
    run_both_modes(d, 8, 6, bf16=True)


@pytest.mark.parametrize("size,h", [(4096, 6), (4096, 4)])
def test_large_square_gemm_sampled_rows_and_checksums(size, h):
    """Config-4 shape in the launch configuration the benchmark times: sampled rows bit-exact
    (including tile-boundary rows), whole-output row/column checksum identities in int64."""
    M = N = K = size
    d = wl.gemm_inputs(4, size + h, M, N, K)
    W, X, mask, ws = d["W"], d["X"], d["mask"], d["w_scale"]
    wh, wlo = oracle.decompose(W, mask, 8, h, True)
    hi, lo = nq.nq_decompose(dev(W), dev(mask), 8, h, True)
    Wd = nq.nq_recompose(hi, lo, N, K, 8, h, True)
    assert torch.equal(Wd, dev(W))
    Xd, wsd = dev(X), dev(ws)
    rng = wl.rng_for(4, 999)
    rows = np.unique(np.concatenate([[0, 127, 128, 129, 255, 256, M - 129, M - 128, M - 1], rng.integers(0, M, 40)]))
    rows_t = torch.from_numpy(rows).cuda()
    for part in (False, True):
        Wref = wh if part else W
        if part:
            acc, y = nq.nq_gemm_part(Xd, hi, N, 8, h, wsd, 0.05, want_acc=True)
        else:
            acc, y = nq.nq_gemm_full(Xd, Wd, wsd, 0.05, want_acc=True)
        nq.nq_device_status()
        ref = oracle.gemm_acc(X[rows], Wref)
        assert np.array_equal(host(acc[rows_t]), ref)
        assert np.array_equal(host(y[rows_t]), oracle.dequant(ref, ws, 0.05, (8 - h) if part else 0))
        # sum_j acc[m, j] = x[m, :] . (sum_j w[j, :]) and sum_m acc[m, j] = (sum_m x[m, :]) . w[j, :]
        acc64 = host(acc).astype(np.int64)
        assert np.array_equal(acc64.sum(axis=1), X.astype(np.int64) @ Wref.astype(np.int64).sum(axis=0))
        assert np.array_equal(acc64.sum(axis=0), Wref.astype(np.int64) @ X.astype(np.int64).sum(axis=0))


def test_rejected_arguments():
    X = torch.zeros((128, 130), dtype=torch.int8, device="cuda")
    W = torch.zeros((64, 130), dtype=torch.int8, device="cuda")
    ws = torch.ones(64, device="cuda")
    with pytest.raises(nq.NqError) as e:
        nq.nq_gemm_full(X, W, ws, 1.0)          # pitch 130 is not a multiple of 16
    assert e.value.status == 3
    acc, y = nq.nq_gemm_full(X[:0], W, ws, 1.0)  # empty M: nothing to do
    assert y.shape == (0, 64)


@pytest.mark.parametrize("acc_plain", [True, False])
def test_one_output_by_tile_stores_the_other_by_ordinary_stores(acc_plain):
    """The two outputs of a launch share a warp's staging block.  With one of them on tile stores (aligned) and the
    other on ordinary stores (pitch not a multiple of 16 bytes) the ordinary path must not overwrite a block that a
    tile store in flight still reads: many chunks per warp, several launches, every value checked."""
    M, N, K = 1030, 1100, 256
    d = wl.gemm_inputs(90, int(acc_plain), M, N, K)
    Xd, Wd, wsd = dev_padded(d["X"]), dev_padded(d["W"]), dev(d["w_scale"])
    acc_ref = oracle.gemm_acc(d["X"], d["W"])
    y_ref = oracle.dequant(acc_ref, d["w_scale"], d["act_scale"], 0)
    for _ in range(4):
        if acc_plain:
            acc = torch.zeros((M, N + 1), dtype=torch.int32, device="cuda")[:, :N]
            y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        else:
            acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
            y = torch.full((M, N + 1), float("nan"), dtype=torch.float32, device="cuda")[:, :N]
        nq.nq_gemm_full(Xd, Wd, wsd, d["act_scale"], acc_out=acc, y_out=y)
        nq.nq_device_status()
        assert np.array_equal(host(acc), acc_ref)
        assert np.array_equal(host(y), y_ref)
