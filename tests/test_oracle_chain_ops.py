"""Pins of the oracle's residual hand-over and pooling (the steps a chained model needs between its layers).  The
paper defines none of them (parity unpinned by the paper); the oracle's arithmetic is pinned here by exactly
representable cases worked out by hand, by the tie and saturation rules, by special cases that reduce to the
plain hand-over, and by float64 / numpy restatements of the definitions."""
import numpy as np

import oracle


def rr(acc, res, res_scale, ws=1.0, sa=1.0, l=0, out=1.0, bias=None, relu=False):
    acc = np.array([acc], dtype=np.int32)
    res = np.array([res], dtype=np.int8)
    w = np.full(acc.shape[1], ws, dtype=np.float32)
    b = None if bias is None else np.full(acc.shape[1], bias, dtype=np.float32)
    return oracle.requant_res(acc, w, sa, l, out, res, res_scale, bias=b, relu=relu)[0].tolist()


def test_residual_is_added_dequantised_before_relu_and_rounding():
    # 10 + 1 * 0.5 = 10.5 -> 10 (tie to even); -10 + 2 * 0.5 = -9 -> ReLU -> 0; 4 - 3 * 0.5 = 2.5 -> 2
    assert rr([10, -10, 4], [1, 2, -3], 0.5, relu=True) == [10, 0, 2]
    # without ReLU the negative survives; 11.5 -> 12
    assert rr([10, -10, 11], [1, 2, 1], 0.5) == [10, -9, 12]
    # the skip path alone can saturate either way
    assert rr([0, 0], [127, -128], 2.0) == [127, -128]


def test_zero_residual_reduces_to_the_plain_hand_over():
    rng = np.random.default_rng(3)
    acc = rng.integers(-(1 << 18), 1 << 18, size=(40, 24)).astype(np.int32)
    ws = rng.uniform(1e-3, 1e-2, 24).astype(np.float32)
    bias = rng.normal(size=24).astype(np.float32)
    zero = np.zeros((40, 24), dtype=np.int8)
    for relu in (False, True):
        a = oracle.requant_res(acc, ws, 0.05, 2, 1.3, zero, 0.7, bias=bias, relu=relu)
        b = oracle.requant(acc, ws, 0.05, 2, 1.3, bias=bias, relu=relu)
        assert np.array_equal(a, b)


def test_residual_order_of_operations_bias_then_skip():
    # acc 1, bias 0.25, skip 3 * 0.25: (1 + 0.25) + 0.75 = 2.0 -> out scale 4 -> 0.5 -> 0 (tie to even)
    assert rr([1], [3], 0.25, bias=0.25, out=4.0) == [0]
    # part-bit scale: acc 3 * 2^2 = 12, + 4 * 0.5 = 14 -> / 4 = 3.5 -> 4
    assert rr([3], [4], 0.5, l=2, out=4.0) == [4]


def test_residual_agrees_with_the_float64_value_up_to_one_step():
    rng = np.random.default_rng(9)
    acc = rng.integers(-(1 << 20), 1 << 20, size=(64, 96)).astype(np.int32)
    res = rng.integers(-128, 128, size=(64, 96)).astype(np.int8)
    ws = rng.uniform(1e-3, 1e-2, 96).astype(np.float32)
    q = oracle.requant_res(acc, ws, 0.05, 1, 2.9, res, 0.031, relu=True).astype(np.int64)
    y64 = np.maximum(acc.astype(np.float64) * 0.05 * ws.astype(np.float64) * 2 + res.astype(np.float64) * 0.031, 0.0) / 2.9
    ref = np.clip(np.rint(y64), -128, 127).astype(np.int64)
    assert np.max(np.abs(q - ref)) <= 1 and np.mean(q == ref) > 0.999


def test_max_pooling_small_case_by_hand():
    # 4 x 4 image holding -8 .. 7 row by row, one channel; 3 x 3 window, stride 2, padding 1
    x = np.arange(-8, 8, dtype=np.int8).reshape(1, 4, 4, 1)
    y = oracle.maxpool_nhwc(x, 3, 2, 1)
    assert y.shape == (1, 2, 2, 1)
    assert y[0, :, :, 0].tolist() == [[-3, -1], [5, 7]]
    # padding never wins: an all-negative image keeps its (negative) maxima
    neg = np.full((1, 3, 3, 2), -100, dtype=np.int8)
    neg[0, 1, 1, 1] = -128
    assert np.all(oracle.maxpool_nhwc(neg, 3, 1, 1)[..., 0] == -100)
    assert oracle.maxpool_nhwc(neg, 1, 1, 0)[0, 1, 1, 1] == -128


def test_max_pooling_against_a_numpy_restatement():
    rng = np.random.default_rng(4)
    x = rng.integers(-128, 128, size=(2, 9, 11, 5)).astype(np.int8)
    k, stride, pad = 3, 2, 1
    padded = np.full((2, 9 + 2 * pad, 11 + 2 * pad, 5), -128, dtype=np.int16)
    padded[:, pad:pad + 9, pad:pad + 11, :] = x
    Ho, Wo = (9 + 2 * pad - k) // stride + 1, (11 + 2 * pad - k) // stride + 1
    ref = np.empty((2, Ho, Wo, 5), dtype=np.int8)
    for p in range(Ho):
        for q in range(Wo):
            ref[:, p, q, :] = padded[:, p * stride:p * stride + k, q * stride:q * stride + k, :].max(axis=(1, 2))
    assert np.array_equal(oracle.maxpool_nhwc(x, k, stride, pad), ref)


def test_global_average_pooling_by_hand_and_against_float64():
    x = np.arange(-8, 8, dtype=np.int8).reshape(1, 4, 4, 1)          # sum -8 over 16 pixels: mean -0.5
    assert oracle.avgpool_requant_nhwc(x, 1.0, 0.25).tolist() == [[-2]]
    assert oracle.avgpool_requant_nhwc(x, 1.0, 1.0).tolist() == [[0]]          # -0.5 -> tie to even -> 0
    assert oracle.avgpool_requant_nhwc(np.full((1, 7, 7, 3), 127, np.int8), 4.0, 1.0).tolist() == [[127, 127, 127]]
    rng = np.random.default_rng(6)
    x = rng.integers(0, 128, size=(3, 7, 7, 64)).astype(np.int8)
    q = oracle.avgpool_requant_nhwc(x, 0.037, 0.021).astype(np.int64)
    ref = np.clip(np.rint(x.astype(np.float64).mean(axis=(1, 2)) * 0.037 / 0.021), -128, 127).astype(np.int64)
    assert np.max(np.abs(q - ref)) <= 1 and np.mean(q == ref) > 0.99
