"""Parity of the codec kernels (decompose / recompose / drop-low / pack / unpack) with the CPU oracle.

Everything here is integer and byte work: the bar is bit-exact, on the packed bytes as well as on
the unpacked weights.  All calls go through the C boundary (ctypes binding).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu

NESTINGS = [(8, h, c) for h in range(1, 8) for c in (1, 0)] + [(6, h, c) for h in range(1, 6) for c in (1, 0)]
# several 128-element groups plus a ragged tail; pitch-aligned and unaligned rows; one row and many
SHAPES = [(5, 147), (64, 576), (256, 256), (3, 4128), (1, 1), (33, 130)]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def rand_weights(rng, shape, n):
    return rng.integers(-(2 ** (n - 1)), 2 ** (n - 1), size=shape).astype(np.int8)


def padded(a, ld):
    """Copy a [rows, cols] array into a device buffer with row pitch ld; returns the strided view."""
    rows, cols = a.shape
    buf = torch.zeros((rows, ld), dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    buf[:, :cols] = dev(a)
    return buf[:, :cols]


@pytest.mark.parametrize("n,h,comp", NESTINGS)
def test_decompose_recompose_drop_low_bit_exact(n, h, comp):
    rng = wl.rng_for(91, n * 100 + h * 2 + comp)
    lb = n - h + comp
    for rows, cols in SHAPES:
        w = rand_weights(rng, (rows, cols), n)
        mask = wl.bernoulli_mask(rng, (rows, cols))
        wh, wl_ = oracle.decompose(w, mask, n, h, bool(comp))
        want_hi, want_lo = oracle.pack_sliced(wh, h), oracle.pack_sliced(wl_, lb)
        for ld in (cols, -(-cols // 16) * 16 + 16):
            w_d, m_d = padded(w, ld), padded(mask, ld)
            hi, lo = nq.nq_decompose(w_d, m_d, n, h, bool(comp))
            assert np.array_equal(host(hi), want_hi), (rows, cols, ld, "hi")
            assert np.array_equal(host(lo), want_lo), (rows, cols, ld, "lo")
            out = torch.full((rows, ld), 77, dtype=torch.int8, device="cuda")
            rec = nq.nq_recompose(hi, lo, rows, cols, n, h, bool(comp), out=out[:, :cols])
            assert np.array_equal(host(rec), oracle.recompose(wh, wl_, n, h))
            assert torch.all(out[:, cols:] == 77)            # nothing written past the row
            if comp:
                assert np.array_equal(host(rec), w)          # exact recomposition
            full = dev(oracle.recompose(wh, wl_, n, h))
            hi2 = nq.nq_drop_low(padded(host(full), ld), lo, n, h, bool(comp))
            want = oracle.pack_sliced(oracle.drop_low(host(full), wl_, n, h), h)
            assert np.array_equal(host(hi2), want)
            if comp:
                assert np.array_equal(host(hi2), want_hi)    # drop_low(recompose(H, L), L) == H


@pytest.mark.parametrize("bits", range(1, 9))
def test_pack_unpack_bit_exact(bits):
    rng = wl.rng_for(92, bits)
    for rows, cols in SHAPES:
        v = rng.integers(-(2 ** (bits - 1)), 2 ** (bits - 1), size=(rows, cols)).astype(np.int8)
        p = nq.nq_pack(dev(v), bits)
        assert np.array_equal(host(p), oracle.pack_sliced(v, bits))
        assert np.array_equal(host(nq.nq_unpack(p, bits, rows, cols)), v)


@pytest.mark.parametrize("n,h,comp", [(8, 6, 1), (8, 4, 1), (8, 5, 0), (8, 7, 1), (6, 4, 1), (8, 1, 1)])
def test_recompose_and_drop_low_on_arbitrary_bytes(n, h, comp):
    """Any byte pattern is a valid packed tensor: the clip of the recomposition and the modular
    behaviour of drop-low must agree with the oracle there too."""
    rng = wl.rng_for(93, n * 10 + h)
    lb = n - h + comp
    rows, cols = 37, 384
    pad = oracle.sliced_padded_rows(rows)
    hi = rng.integers(0, 256, size=(pad, oracle.sliced_row_bytes(cols, h)), dtype=np.uint8)
    lo = rng.integers(0, 256, size=(pad, oracle.sliced_row_bytes(cols, lb)), dtype=np.uint8)
    wh, wl_ = oracle.unpack_sliced(hi, rows, cols, h), oracle.unpack_sliced(lo, rows, cols, lb)
    got = host(nq.nq_recompose(dev(hi), dev(lo), rows, cols, n, h, bool(comp)))
    assert np.array_equal(got, oracle.recompose(wh, wl_, n, h))
    w = rand_weights(rng, (rows, cols), n)
    got_hi = host(nq.nq_drop_low(dev(w), dev(lo), n, h, bool(comp)))
    want = oracle.drop_low(w, wl_, n, h)
    assert np.array_equal(got_hi, oracle.pack_sliced(want, h))     # padding rows and columns included: zero fields


def test_paper_invariants_on_the_gpu_at_config1_size():
    c = wl.config1()
    W, mask = c["W"], c["mask"]
    hi, lo = nq.nq_decompose(dev(W), dev(mask), 8, 6, True)
    wh = host(nq.nq_unpack(hi, 6, 256, 256))
    wlow = host(nq.nq_unpack(lo, 3, 256, 256))
    assert wh.min() >= -32 and wh.max() <= 31 and wlow.min() >= -3 and wlow.max() <= 3
    x = W.astype(np.float64) / 4
    assert np.array_equal(wh, np.clip(np.where(mask == 1, np.ceil(x), np.floor(x)), -32, 31))
    assert np.array_equal(host(nq.nq_recompose(hi, lo, 256, 256, 8, 6, True)), W)
    # the paper's worked example through the kernels: -67 in INT(8|4), BitShift rounding
    w = np.full((1, 128), -67, dtype=np.int8)
    hi4, lo5 = nq.nq_decompose(dev(w), dev(np.zeros_like(w, dtype=np.uint8)), 8, 4, True)
    assert host(nq.nq_unpack(hi4, 4, 1, 128))[0, 0] == -5 and host(nq.nq_unpack(lo5, 5, 1, 128))[0, 0] == 13
    hi4c, lo4c = nq.nq_decompose(dev(w), dev(np.zeros_like(w, dtype=np.uint8)), 8, 4, False)
    assert host(nq.nq_unpack(lo4c, 4, 1, 128))[0, 0] == 7
    assert host(nq.nq_recompose(hi4c, lo4c, 1, 128, 8, 4, False))[0, 0] == -73


def test_batched_page_in_and_page_out_match_the_single_tensor_calls():
    rng = wl.rng_for(94)
    shapes = [(64, 576), (128, 64), (7, 147), (256, 1152), (1000, 512), (64, 64)]
    n, h = 8, 6
    tensors, originals = [], []
    for rows, cols in shapes:
        w = rand_weights(rng, (rows, cols), n)
        mask = wl.bernoulli_mask(rng, (rows, cols))
        ld = -(-cols // 16) * 16
        hi, lo = nq.nq_decompose(padded(w, ld), padded(mask, ld), n, h, True)
        out = torch.zeros((rows, ld), dtype=torch.int8, device="cuda")
        tensors.append({"w_int": out[:, :cols], "packed_high": torch.zeros_like(hi), "packed_low": lo})
        originals.append((w, hi))
    plan = nq.nq_batch_plan(tensors)
    for t, (w, hi) in zip(tensors, originals):
        t["packed_high"].copy_(hi)
    nq.nq_recompose_batched(plan, n, h, True)
    for t, (w, hi) in zip(tensors, originals):
        assert np.array_equal(host(t["w_int"]), w)
        t["packed_high"].zero_()
    nq.nq_drop_low_batched(plan, n, h, True)
    for t, (w, hi) in zip(tensors, originals):
        assert torch.equal(t["packed_high"], hi)


def test_empty_and_rejected_inputs():
    e = torch.empty((0, 128), dtype=torch.int8, device="cuda")
    m = torch.empty((0, 128), dtype=torch.uint8, device="cuda")
    hi, lo = nq.nq_decompose(e, m, 8, 6, True)
    assert hi.shape[0] == 0 and lo.shape[0] == 0
    w = torch.zeros((4, 128), dtype=torch.int8, device="cuda")
    mk = torch.zeros((4, 128), dtype=torch.uint8, device="cuda")
    with pytest.raises(nq.NqError):
        nq.nq_decompose(w, mk, 8, 8, True)
    hi, lo = nq.nq_decompose(w, mk, 8, 6, True)
    off = torch.zeros(hi.numel() + 16, dtype=torch.uint8, device="cuda")[1:1 + hi.numel()].view(hi.shape)
    with pytest.raises(nq.NqError) as ei:
        nq.nq_recompose(off, lo, 4, 128, 8, 6, True)
    assert ei.value.status == 3


def test_large_tensor_sampled_against_the_oracle():
    """Full-size page-in at the launch shape the benchmark uses (8192 x 8192), checked on sampled rows."""
    rng = wl.rng_for(95)
    rows = cols = 8192
    w = wl.clipped_normal_int8(rng, (rows, cols), 40.0)
    mask = wl.bernoulli_mask(rng, (rows, cols))
    hi, lo = nq.nq_decompose(dev(w), dev(mask), 8, 5, True)
    rec = nq.nq_recompose(hi, lo, rows, cols, 8, 5, True)
    assert torch.equal(rec, dev(w))
    # the packed bytes of three whole row blocks (a row block's 128 x 128 blocks are contiguous in storage) ...
    for rb in (0, 17, rows // 128 - 1):
        band = slice(rb * 128, rb * 128 + 128)
        wh, wl_ = oracle.decompose(w[band], mask[band], 8, 5, True)
        assert np.array_equal(host(hi[band]), oracle.pack_sliced(wh, 5))
        assert np.array_equal(host(lo[band]), oracle.pack_sliced(wl_, 4))
    # ... and the field values of sampled rows anywhere
    sample = np.unique(np.concatenate([[0, 1, 127, 128, rows - 1], rng.integers(0, rows, 40)]))
    wh, wl_ = oracle.decompose(w[sample], mask[sample], 8, 5, True)
    idx = torch.from_numpy(sample).cuda()
    assert np.array_equal(host(nq.nq_unpack(hi, 5, rows, cols)[idx]), wh)
    assert np.array_equal(host(nq.nq_unpack(lo, 4, rows, cols)[idx]), wl_)
