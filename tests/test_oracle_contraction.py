"""Pins for the oracle's integer GEMM, dequantisation and convolution.

The paper gives no worked numbers for the integer layer, so the pins are: brute force in pure Python
on tiny inputs, an exact float64 library matmul / conv2d (a different routine from the oracle's
loops), closed forms for special inputs, and the identity Eq. 5 implies between the two modes.
"""
import numpy as np
import pytest
import torch

import oracle


def _rand_i8(rng, shape, lo=-128, hi=128):
    return rng.integers(lo, hi, size=shape).astype(np.int8)


def test_gemm_brute_force_tiny():
    rng = np.random.default_rng(1)
    x, w = _rand_i8(rng, (3, 5)), _rand_i8(rng, (4, 5))
    acc = oracle.gemm_acc(x, w)
    for m in range(3):
        for j in range(4):
            assert int(acc[m, j]) == sum(int(x[m, k]) * int(w[j, k]) for k in range(5))


def test_gemm_is_not_transposed_and_not_symmetric():
    x = np.array([[1, 2, 3]], dtype=np.int8)
    w = np.array([[1, 0, 0], [0, 0, 1]], dtype=np.int8)      # one-hot rows pick columns of x
    assert oracle.gemm_acc(x, w).tolist() == [[1, 3]]


@pytest.mark.parametrize("M,N,K", [(17, 33, 129), (64, 256, 256), (5, 7, 4099)])
def test_gemm_against_exact_float64_library_matmul(M, N, K):
    rng = np.random.default_rng(M * N + K)
    x, w = _rand_i8(rng, (M, K)), _rand_i8(rng, (N, K))
    want = x.astype(np.float64) @ w.astype(np.float64).T      # exact: |sum| < 2^53
    assert np.array_equal(oracle.gemm_acc(x, w).astype(np.float64), want)


def test_gemm_extreme_values_do_not_overflow_int32():
    K = 16384
    x = np.full((1, K), -128, dtype=np.int8)
    w = np.full((1, K), -128, dtype=np.int8)
    assert int(oracle.gemm_acc(x, w)[0, 0]) == K * 128 * 128


def test_gemm_closed_forms():
    rng = np.random.default_rng(3)
    w = _rand_i8(rng, (9, 40))
    ones = np.ones((2, 40), dtype=np.int8)
    assert np.array_equal(oracle.gemm_acc(ones, w)[0], w.astype(np.int32).sum(axis=1))
    assert not oracle.gemm_acc(_rand_i8(rng, (4, 40)), np.zeros((9, 40), np.int8)).any()


@pytest.mark.parametrize("h", [3, 4, 5, 6, 7])
def test_full_bit_equals_scaled_part_bit_plus_low_contribution(h):
    # Eq. 5 under the contraction: X W_int^T = 2^l X W_high^T + X W_low^T, exactly
    rng = np.random.default_rng(h)
    w = _rand_i8(rng, (24, 96))
    mask = rng.integers(0, 2, size=w.shape).astype(np.uint8)
    x = _rand_i8(rng, (10, 96))
    wh, wl = oracle.decompose(w, mask, 8, h)
    full = oracle.gemm_acc(x, oracle.recompose(wh, wl, 8, h)).astype(np.int64)
    part = oracle.gemm_acc(x, wh).astype(np.int64)
    low = oracle.gemm_acc(x, wl).astype(np.int64)
    assert np.array_equal(full, (part << (8 - h)) + low)


def test_dequant_fp32_rounding_order_and_fp64_reference():
    rng = np.random.default_rng(5)
    acc = rng.integers(-2 ** 27, 2 ** 27, size=(6, 11)).astype(np.int32)
    ws = rng.uniform(1e-3, 1e-2, size=11).astype(np.float32)
    sa = np.float32(0.05)
    for l in (0, 2, 4):
        y, yref = oracle.dequant(acc, ws, float(sa), l, want_ref=True)
        scale = (sa * ws).astype(np.float32) * np.float32(2 ** l)        # numpy rounds each op to fp32
        want = acc.astype(np.float32) * scale
        assert y.dtype == np.float32 and np.array_equal(y, want)
        exact = acc.astype(np.float64) * float(sa) * ws.astype(np.float64) * 2 ** l
        assert np.allclose(yref, exact, rtol=1e-15)
        assert np.max(np.abs(y - exact)) <= 4e-7 * np.max(np.abs(exact))
    b = rng.normal(size=11).astype(np.float32)
    yb = oracle.dequant(acc, ws, float(sa), 0, bias=b)
    assert np.array_equal(yb, acc.astype(np.float32) * (sa * ws).astype(np.float32) + b)


def test_part_bit_dequant_is_the_inflated_scale_of_eq9():
    # s_high = s * 2^l: dequantising w_high with l_shift = l equals dequantising (w_high * 2^l) with l_shift = 0
    acc = np.array([[12345, -678]], dtype=np.int32)
    ws = np.array([0.004, 0.009], dtype=np.float32)
    a = oracle.dequant(acc, ws, 0.05, 3)
    b = oracle.dequant(acc * 8, ws, 0.05, 0)
    assert np.array_equal(a, b)


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(size=4096).astype(np.float32) * 100,
                        np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 0.0], dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16_bits(x), want)


def test_conv_brute_force_tiny():
    rng = np.random.default_rng(2)
    B, C, H, W, Co, R, S, st, pad = 1, 2, 5, 4, 3, 3, 3, 2, 1
    x, w = _rand_i8(rng, (B, C, H, W)), _rand_i8(rng, (Co, C, R, S))
    acc = oracle.conv_acc(x, w, st, pad)
    Ho, Wo = (H + 2 * pad - R) // st + 1, (W + 2 * pad - S) // st + 1
    assert acc.shape == (B, Co, Ho, Wo)
    for co in range(Co):
        for p in range(Ho):
            for q in range(Wo):
                s = 0
                for ci in range(C):
                    for r in range(R):
                        for t in range(S):
                            ih, iw = p * st - pad + r, q * st - pad + t
                            if 0 <= ih < H and 0 <= iw < W:
                                s += int(x[0, ci, ih, iw]) * int(w[co, ci, r, t])
                assert int(acc[0, co, p, q]) == s


@pytest.mark.parametrize("cfg", [(2, 3, 9, 9, 4, 7, 2, 3), (2, 8, 6, 7, 5, 3, 1, 1), (1, 16, 8, 8, 8, 1, 2, 0),
                                 (2, 4, 7, 7, 6, 3, 2, 1)])
def test_conv_against_float64_library_conv2d(cfg):
    B, C, H, W, Co, R, st, pad = cfg
    rng = np.random.default_rng(sum(cfg))
    x, w = _rand_i8(rng, (B, C, H, W)), _rand_i8(rng, (Co, C, R, R))
    want = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(),
                                      stride=st, padding=pad).numpy()
    got = oracle.conv_acc(x, w, st, pad)
    assert got.shape == want.shape and np.array_equal(got.astype(np.float64), want)
    pix = np.array([[0, 0, 0], [B - 1, got.shape[2] - 1, got.shape[3] - 1], [0, 1, 0]])
    sub = oracle.conv_acc_pixels(x, w, st, pad, pix)
    for i, (b, p, q) in enumerate(pix):
        assert np.array_equal(sub[i], got[b, :, p, q])


def test_pointwise_conv_is_the_gemm():
    rng = np.random.default_rng(4)
    x, w = _rand_i8(rng, (2, 12, 5, 6)), _rand_i8(rng, (7, 12, 1, 1))
    conv = oracle.conv_acc(x, w, 1, 0)                                     # [B, Co, H, W]
    gemm = oracle.gemm_acc(x.transpose(0, 2, 3, 1).reshape(-1, 12), w.reshape(7, 12))
    assert np.array_equal(conv.transpose(0, 2, 3, 1).reshape(-1, 7), gemm)


def test_conv_of_all_ones_without_padding_gives_weight_sums():
    rng = np.random.default_rng(6)
    w = _rand_i8(rng, (5, 3, 3, 3))
    x = np.ones((1, 3, 6, 6), dtype=np.int8)
    acc = oracle.conv_acc(x, w, 1, 0)
    assert np.array_equal(acc[0, :, 2, 1], w.astype(np.int32).sum(axis=(1, 2, 3)))
    # with padding, the corner loses the taps that fall outside the image
    accp = oracle.conv_acc(x, w, 1, 1)
    assert np.array_equal(accp[0, :, 0, 0], w[:, :, 1:, 1:].astype(np.int32).sum(axis=(1, 2, 3)))
