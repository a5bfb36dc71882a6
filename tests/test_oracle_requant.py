"""Pins of the oracle's requantisation (a layer's accumulators -> INT8 activations of the next layer).  The paper
does not define this step (parity unpinned by the paper); the oracle's arithmetic is pinned here by exactly
representable cases worked out by hand, by the tie and saturation rules of Eq. 1, and by the float64 value."""
import numpy as np

import oracle


def rq(acc, ws=1.0, sa=1.0, l=0, out=1.0, bias=None, relu=False):
    acc = np.array([acc], dtype=np.int32)
    w = np.full(acc.shape[1], ws, dtype=np.float32)
    b = None if bias is None else np.full(acc.shape[1], bias, dtype=np.float32)
    return oracle.requant(acc, w, sa, l, out, bias=b, relu=relu)[0].tolist()


def test_identity_scales_give_the_clipped_accumulator():
    assert rq([0, 1, -1, 127, 128, -128, -129, 100000, -100000]) == [0, 1, -1, 127, 127, -128, -128, 127, -128]


def test_relu_zeroes_negatives_before_the_rounding():
    assert rq([-5, -1, 0, 1, 300], relu=True) == [0, 0, 0, 1, 127]


def test_ties_go_to_the_even_integer():
    # act_scale 0.5: values k + 0.5 exactly
    assert rq([1, 3, 5, 7, -1, -3, -5], sa=0.5) == [0, 2, 2, 4, 0, -2, -2]
    # output scale 4: 10 / 4 = 2.5 -> 2, 14 / 4 = 3.5 -> 4, 6 / 4 = 1.5 -> 2
    assert rq([10, 14, 6, 9, 11], out=4.0) == [2, 4, 2, 2, 3]


def test_part_bit_scale_carries_two_to_the_l():
    assert rq([3, -3], l=2) == [12, -12]
    assert rq([3, -3], l=3, out=8.0) == [3, -3]


def test_bias_is_added_before_relu_and_rounding():
    assert rq([0, 0], bias=2.5) == [2, 2]
    assert rq([1, -10], bias=2.5, relu=True) == [4, 0]          # 3.5 -> 4; -7.5 -> relu -> 0


def test_agrees_with_the_float64_value_up_to_one_step_and_mostly_exactly():
    rng = np.random.default_rng(5)
    acc = rng.integers(-(1 << 20), 1 << 20, size=(64, 96)).astype(np.int32)
    ws = rng.uniform(1e-3, 1e-2, 96).astype(np.float32)
    sa, out_scale, l = 0.05, 3.7, 2
    q = oracle.requant(acc, ws, sa, l, out_scale, relu=True).astype(np.int64)
    y64 = np.maximum(acc.astype(np.float64) * sa * ws.astype(np.float64) * (1 << l), 0.0) / out_scale
    ref = np.clip(np.rint(y64), -128, 127).astype(np.int64)
    assert np.max(np.abs(q - ref)) <= 1
    assert np.mean(q == ref) > 0.999
