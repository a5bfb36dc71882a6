"""The large square nested GEMM sweep at its two large sizes, M = N = K in {8192, 16384}, against the oracle.

These are the sizes that carry almost all of the benchmark's integer operations.  Every launch here is the one
the benchmark makes (same entry point, same pointers' alignment, the CTA-pair kernel), and is checked three ways:
  - about fifty sampled rows -- first and last rows of the first, second and last 256-row tile, plus random ones --
    bit for bit on the INT32 accumulators and on the fp32 output (Eq. 2 full-bit, Eq. 9 part-bit);
  - the whole accumulator through two exact identities in int64,
        sum_j acc[m, j] = x[m, :] . (sum_j w[j, :])     and     sum_m acc[m, j] = (sum_m x[m, :]) . w[j, :];
  - a second launch that writes bf16 only (no accumulator output: the epilogue the benchmark times), on the same
    sampled rows against the round-to-nearest-even bf16 of the oracle's fp32 value.
Modes: full-bit on the weights the GPU recomposed itself; part-bit for h = 4 (fields read straight from the packed
matrix) and h = 5, 6, 7 (ring of packed tiles); at 8192 also the nested full-bit GEMM (Eq. 5 inside the kernel)
for h = 6 and h = 3.  The packed tensors the GPU wrote are compared with the oracle's packing byte for byte.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ACT = 0.05


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def sampled_rows(M, seed):
    rng = wl.rng_for(4, seed)
    fixed = [0, 1, 127, 128, 255, 256, 257, 383, 511, 512, M - 256, M - 255, M - 129, M - 128, M - 2, M - 1]
    return np.unique(np.concatenate([fixed, rng.integers(0, M, 36)]))


def int64_row_dot(A, v, block=2048):
    """A (int8 [R, K]) times v (int64 [K]) in int64, in row blocks so that the int64 copy of A stays small."""
    out = np.empty(A.shape[0], dtype=np.int64)
    for r0 in range(0, A.shape[0], block):
        out[r0:r0 + block] = A[r0:r0 + block].astype(np.int64) @ v
    return out


def check_launch(run, X, Wref, ws, l_shift, rows, rows_t):
    """run(want_acc, y_dtype) -> (acc, y).  Wref: the int8 matrix the mode contracts with, per the oracle."""
    acc, y = run(True, torch.float32)
    nq.nq_device_status()
    ref = oracle.gemm_acc(X[rows], Wref)
    assert np.array_equal(host(acc[rows_t]), ref), "sampled accumulator rows differ"
    y_ref = oracle.dequant(ref, ws, ACT, l_shift)
    got = host(y[rows_t])
    assert np.max(np.abs(got.astype(np.float64) - y_ref)) <= 1e-5 * np.max(np.abs(y_ref))
    assert np.array_equal(got, y_ref), "sampled fp32 rows differ"
    # whole-output identities; the two sums of the accumulator are taken on the device in int64
    row_sum = host(acc.sum(dim=1, dtype=torch.int64))
    col_sum = host(acc.sum(dim=0, dtype=torch.int64))
    w_col = Wref.sum(axis=0, dtype=np.int64)
    x_col = X.sum(axis=0, dtype=np.int64)
    assert np.array_equal(row_sum, int64_row_dot(X, w_col)), "row checksums differ"
    assert np.array_equal(col_sum, int64_row_dot(Wref, x_col)), "column checksums differ"
    del acc, y
    # the benchmark's launch: bf16 out, no accumulator output
    _, yb = run(False, torch.bfloat16)
    nq.nq_device_status()
    got16 = host(yb[rows_t].view(torch.int16)).view(np.uint16)
    assert np.array_equal(got16, oracle.f32_to_bf16_bits(y_ref)), "sampled bf16 rows differ"


@pytest.mark.parametrize("size", [8192, 16384])
def test_config4_large_sizes_every_mode(size):
    M = N = K = size
    d = wl.gemm_inputs(4, size, M, N, K)
    W, X, mask, ws = d["W"], d["X"], d["mask"], d["w_scale"]
    Xd, Wd, md, wsd = dev(X), dev(W), dev(mask), dev(ws)
    rows = sampled_rows(M, size)
    rows_t = torch.from_numpy(rows).cuda()
    first = True
    for h in (4, 5, 6, 7):
        l = 8 - h
        wh, wlo = oracle.decompose(W, mask, 8, h, True)
        hi, lo = nq.nq_decompose(Wd, md, 8, h, True)
        assert np.array_equal(host(hi), oracle.pack_sliced(wh, h)), "packed w_high differs"
        assert np.array_equal(host(lo), oracle.pack_sliced(wlo, l + 1)), "packed w_low differs"
        if first:                                    # full-bit once per size, on the GPU's own recomposition
            w_rec = nq.nq_recompose(hi, lo, N, K, 8, h, True)
            assert torch.equal(w_rec, Wd)
            assert torch.equal(nq.nq_drop_low(w_rec, lo, 8, h, True), hi)
            check_launch(lambda acc, ydt: nq.nq_gemm_full(Xd, w_rec, wsd, ACT, want_acc=acc, y_dtype=ydt),
                         X, W, ws, 0, rows, rows_t)
            del w_rec
            first = False
        check_launch(lambda acc, ydt: nq.nq_gemm_part(Xd, hi, N, 8, h, wsd, ACT, want_acc=acc, y_dtype=ydt),
                     X, wh, ws, l, rows, rows_t)
        del hi, lo
    if size == 8192:
        for h in (6, 3):                             # h = 3: the narrow field's 1-bit slice rides in the ring tile
            wh, wlo = oracle.decompose(W, mask, 8, h, True)
            hi, lo = nq.nq_decompose(Wd, md, 8, h, True)
            w_full = oracle.recompose(wh, wlo, 8, h)
            assert np.array_equal(w_full, W)
            check_launch(lambda acc, ydt: nq.nq_gemm_nested(Xd, hi, lo, N, 8, h, wsd, ACT, want_acc=acc, y_dtype=ydt),
                         X, w_full, ws, 0, rows, rows_t)
            del hi, lo
