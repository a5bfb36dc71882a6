"""Seeded random shapes through both GEMM modes against the oracle, and repeated launches of the large kernels that
must give the same bytes every time (a race between the producer, unpack, MMA and epilogue roles would not)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def padded(a):
    rows, cols = a.shape
    ld = -(-cols // 16) * 16
    buf = torch.zeros((rows, ld), dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    buf[:, :cols] = dev(a)
    return buf[:, :cols]


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_both_modes(seed):
    rng = wl.rng_for(98, seed)
    for _ in range(6):
        M, N, K = int(rng.integers(1, 700)), int(rng.integers(1, 700)), int(rng.integers(1, 900))
        h = int(rng.integers(1, 8))
        bf16 = bool(rng.integers(0, 2))
        d = wl.gemm_inputs(98, seed * 100 + M + N + K, M, N, K)
        wh, wlo = oracle.decompose(d["W"], d["mask"], 8, h, True)
        hi, lo = nq.nq_decompose(padded(d["W"]), padded(d["mask"]), 8, h, True)
        Xd, wsd = padded(d["X"]), dev(d["w_scale"])
        ydt = torch.bfloat16 if bf16 else torch.float32
        for part in (False, True):
            if part:
                acc, y = nq.nq_gemm_part(Xd, hi, N, 8, h, wsd, d["act_scale"], want_acc=True, y_dtype=ydt)
                ref = oracle.gemm_acc(d["X"], wh)
            else:
                acc, y = nq.nq_gemm_full(Xd, padded(d["W"]), wsd, d["act_scale"], want_acc=True, y_dtype=ydt)
                ref = oracle.gemm_acc(d["X"], d["W"])
            assert np.array_equal(acc.cpu().numpy(), ref), (M, N, K, h, part)
            yref = oracle.dequant(ref, d["w_scale"], d["act_scale"], (8 - h) if part else 0)
            if bf16:
                assert np.array_equal(y.view(torch.int16).cpu().numpy().view(np.uint16), oracle.f32_to_bf16_bits(yref))
            else:
                assert np.array_equal(y.cpu().numpy(), yref), (M, N, K, h, part)
        if h >= 2:
            # nested full-bit mode: the full-bit result again, rebuilt from the two packed parts
            acc, y = nq.nq_gemm_nested(Xd, hi, lo, N, 8, h, wsd, d["act_scale"], want_acc=True, y_dtype=ydt)
            ref = oracle.gemm_acc(d["X"], oracle.recompose(wh, wlo, 8, h))
            assert np.array_equal(acc.cpu().numpy(), ref), (M, N, K, h, "nested")
            if not bf16:
                assert np.array_equal(y.cpu().numpy(), oracle.dequant(ref, d["w_scale"], d["act_scale"], 0)), (M, N, K, h)
        nq.nq_device_status()


@pytest.mark.parametrize("h", [3, 5, 6])
def test_repeated_nested_launches_give_identical_bytes(h):
    M, N, K = 2304, 2048, 3072
    g = torch.Generator(device="cuda")
    g.manual_seed(40 + h)
    X = torch.randint(-128, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
    W = torch.randint(-128, 128, (N, K), dtype=torch.int8, device="cuda", generator=g)
    mask = torch.randint(0, 2, (N, K), dtype=torch.uint8, device="cuda", generator=g)
    hi, lo = nq.nq_decompose(W, mask, 8, h, True)
    ws = torch.rand(N, device="cuda", generator=g) * 1e-2 + 1e-3
    first_f, _ = nq.nq_gemm_full(X, W, ws, 0.05, want_acc=True, y_dtype=None)
    for _ in range(15):
        again, _ = nq.nq_gemm_nested(X, hi, lo, N, 8, h, ws, 0.05, want_acc=True, y_dtype=None)
        assert torch.equal(again, first_f)
    nq.nq_device_status()


@pytest.mark.parametrize("h", [4, 6, 7])
def test_repeated_launches_give_identical_bytes(h):
    M, N, K = 2304, 2048, 3072            # CTA-pair kernel, several waves, 24 K-blocks
    g = torch.Generator(device="cuda")
    g.manual_seed(h)
    X = torch.randint(-128, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
    lim = 1 << (h - 1)
    Wh = torch.randint(-lim, lim, (N, K), dtype=torch.int8, device="cuda", generator=g)
    hi = nq.nq_pack(Wh, h)
    ws = torch.rand(N, device="cuda", generator=g) * 1e-2 + 1e-3
    first_p, _ = nq.nq_gemm_part(X, hi, N, 8, h, ws, 0.05, want_acc=True, y_dtype=None)
    first_f, _ = nq.nq_gemm_full(X, Wh, ws, 0.05, want_acc=True, y_dtype=None)
    assert torch.equal(first_p, first_f)                  # both modes see the same integer weights here
    for _ in range(15):
        again_p, _ = nq.nq_gemm_part(X, hi, N, 8, h, ws, 0.05, want_acc=True, y_dtype=None)
        again_f, _ = nq.nq_gemm_full(X, Wh, ws, 0.05, want_acc=True, y_dtype=None)
        assert torch.equal(again_p, first_p) and torch.equal(again_f, first_f)
    nq.nq_device_status()
