"""Parity of the nested full-bit GEMM (weights rebuilt from the two packed parts inside the kernel).

Expected values: the oracle's recomposition (Eq. 5) followed by its plain integer GEMM and dequantisation.
INT32 accumulators bit-exact, fp32 outputs equal and within 1e-5 of the largest output, bf16 outputs equal to
the round-to-nearest-even bf16 of the oracle's fp32 value.  The packed operands come from the oracle's own
decomposition and packing in one half of the cases and from the GPU's ``nq_decompose`` in the other.
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
    rows, cols = a.shape
    ld = -(-cols // multiple) * multiple
    buf = torch.zeros((rows, ld), dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    buf[:, :cols] = dev(a)
    return buf[:, :cols]


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def expected(d, n, h, bias=None):
    wh, wlo = oracle.decompose(d["W"], d["mask"], n, h, True)
    w_int = oracle.recompose(wh, wlo, n, h)
    assert np.array_equal(w_int, d["W"])           # compensated: Eq. 5 is exact
    acc = oracle.gemm_acc(d["X"], w_int)
    y = oracle.dequant(acc, d["w_scale"], d["act_scale"], 0, bias=bias)
    return wh, wlo, acc, y


def run_nested(d, n, h, bias=None, bf16=False, packed_by_oracle=False):
    N, K = d["W"].shape
    wh, wlo, acc_ref, y_ref = expected(d, n, h, bias)
    if packed_by_oracle:
        hi, lo = dev(oracle.pack_sliced(wh, h)), dev(oracle.pack_sliced(wlo, n - h + 1))
    else:
        hi, lo = nq.nq_decompose(dev_padded(d["W"]), dev_padded(d["mask"]), n, h, True)
    bd = None if bias is None else dev(bias)
    acc, y = nq.nq_gemm_nested(dev_padded(d["X"]), hi, lo, N, n, h, dev(d["w_scale"]), d["act_scale"], bias=bd,
                               want_acc=True, y_dtype=torch.bfloat16 if bf16 else torch.float32)
    nq.nq_device_status()
    assert np.array_equal(host(acc), acc_ref), "int32 accumulators differ"
    if bf16:
        assert np.array_equal(host(y.view(torch.int16)).view(np.uint16), oracle.f32_to_bf16_bits(y_ref))
    else:
        got = host(y)
        assert np.max(np.abs(got.astype(np.float64) - y_ref)) <= REL_TOL * np.max(np.abs(y_ref))
        assert np.array_equal(got, y_ref)


@pytest.mark.parametrize("h", [2, 3, 4, 5, 6, 7])
def test_every_int8_nesting(h):
    d = wl.gemm_inputs(95, h, 300, 520, 640)
    run_nested(d, 8, h, packed_by_oracle=(h % 2 == 0))


@pytest.mark.parametrize("h", [2, 3, 4, 5])
def test_every_int6_nesting(h):
    rng = wl.rng_for(96, h)
    d = wl.gemm_inputs(96, h, 260, 300, 512)
    d["W"] = wl.uniform_int8(rng, (300, 512), -32, 31)
    d["X"] = wl.uniform_int8(rng, (260, 512), -32, 31)
    bias = rng.normal(size=300).astype(np.float32)
    run_nested(d, 6, h, bias=bias, packed_by_oracle=(h % 2 == 1))


# several tiles in every direction, ragged tails, one row, fewer rows or columns than half a tile
SHAPES = [(64, 256, 256), (130, 200, 147), (3500, 1100, 1100), (1, 1000, 512), (257, 96, 4099), (7, 24, 32)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_ragged_shapes(M, N, K):
    d = wl.gemm_inputs(97, M + N + K, M, N, K)
    run_nested(d, 8, 5)
    run_nested(d, 8, 4, bf16=True, packed_by_oracle=True)


def test_extreme_weights_and_every_field_value():
    # all 256 INT8 weight values in every column phase, both rounding directions, extreme activations
    n, h = 8, 6
    W = ((np.arange(256)[:, None] + np.arange(640)[None, :]) % 256 - 128).astype(np.int8)
    rng = wl.rng_for(98)
    mask = wl.bernoulli_mask(rng, W.shape)
    X = wl.uniform_int8(rng, (384, 640))
    X[0, :] = -128
    X[1, :] = 127
    d = {"W": W, "X": X, "mask": mask, "w_scale": wl.channel_scales(rng, 256), "act_scale": 0.03}
    run_nested(d, n, h)
    run_nested(d, n, 2, packed_by_oracle=True)
    run_nested(d, n, 7)


def test_matches_full_bit_gemm_on_the_recomposed_tensor():
    d = wl.gemm_inputs(99, 0, 1024, 768, 1152)
    n, h = 8, 4
    hi, lo = nq.nq_decompose(dev(d["W"]), dev(d["mask"]), n, h, True)
    X, ws = dev(d["X"]), dev(d["w_scale"])
    Wfull = nq.nq_recompose(hi, lo, 768, 1152, n, h, True)
    acc_f, y_f = nq.nq_gemm_full(X, Wfull, ws, 0.05, want_acc=True)
    acc_n, y_n = nq.nq_gemm_nested(X, hi, lo, 768, n, h, ws, 0.05, want_acc=True)
    assert torch.equal(acc_f, acc_n) and torch.equal(y_f, y_n)


def test_unsupported_nestings_and_empty_problems():
    X = torch.zeros((16, 128), dtype=torch.int8, device="cuda")
    p = torch.zeros((16, 16 * 9), dtype=torch.uint8, device="cuda")
    ws = torch.ones(16, device="cuda")
    for n, h in [(8, 1), (7, 4), (6, 1), (6, 6), (8, 8)]:
        with pytest.raises(nq.NqError):
            nq.nq_gemm_nested(X, p, p, 16, n, h, ws, 1.0)
    acc, y = nq.nq_gemm_nested(X[:0], p, p, 16, 8, 4, ws, 1.0, want_acc=True)
    assert acc.shape == (0, 16) and y.shape == (0, 16)
    # a packed operand that is not 16-byte aligned is refused before anything is launched
    big = torch.zeros(16 * 16 * 9 + 16, dtype=torch.uint8, device="cuda")
    off = (-big.data_ptr()) % 16 + 4
    skew = big[off:off + 16 * 16 * 5].view(16, 80)
    with pytest.raises(nq.NqError):
        nq.nq_gemm_nested(X, p[:, :64].contiguous(), skew, 16, 8, 4, ws, 1.0)
    nq.nq_device_status()
