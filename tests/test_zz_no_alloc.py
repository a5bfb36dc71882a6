"""The allocation-free convolution entry point against the ordinary one.

Some users of this library run where device memory cannot be allocated on the fly (an inference plug-in
that only ever sees the buffers its host application hands it, a control loop that must stay clear of the
allocator).  nq_conv_implicit_gemm_static serves them: same inputs and outputs, no workspace, staging
through an array built into the library.  This file checks, through the C boundary, that it returns
exactly what nq_conv_implicit_gemm returns -- bit-exact INT32 accumulators and identical fp32 outputs,
the bar the other convolution tests use -- on two calls in a row that reuse the shared array, that its result is
the CPU oracle's direct convolution, that the device's free memory is the same before and after a call, and that
a layer too large for the array is refused.  It is named so that pytest collects it after every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _layer_tensors(L, batch, seed):
    d = wl.conv_layer_inputs(73, seed, L, batch)
    ldw = -(-L.K // 16) * 16
    w = _dev(wl.oihw_to_ohwi_matrix(d["W"], ldw))[:, :L.K]
    m = _dev(wl.oihw_to_ohwi_matrix(d["mask"], ldw))[:, :L.K]
    hi, _ = nq.nq_decompose(w, m, 8, 6, True)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)      # NCHW: needs staging
    return desc, _dev(d["X"]), w, hi, _dev(d["w_scale"]), d["act_scale"]


def _compare(L, batch, seed, part):
    desc, x, w, hi, ws, sa = _layer_tensors(L, batch, seed)
    assert 0 < nq.nq_conv_workspace_bytes(desc) <= nq.NQ_CONV_STATIC_SCRATCH_BYTES
    weights = hi if part else w
    acc_ref, y_ref, _ = nq.nq_conv_implicit_gemm(x, weights, desc, ws, sa, part_bit=part, n_bits=8, h_bits=6, want_acc=True)
    acc = torch.full_like(acc_ref, -1)
    y = torch.full_like(y_ref, float("nan"))
    nq.nq_conv_implicit_gemm_static(x, weights, desc, ws, sa, acc, y, part_bit=part, n_bits=8, h_bits=6)
    nq.nq_device_status()
    assert torch.equal(acc, acc_ref)
    assert torch.equal(y, y_ref)
    assert float((y - y_ref).abs().max()) <= 1e-5 * float(y_ref.abs().max())


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    big = wl.ConvLayer("c64", 64, 28, 28, 64, 3, 3, 1, 1)          # 401 KiB of staging (NCHW -> NHWC copy)
    small = wl.ConvLayer("stem", 3, 20, 20, 32, 7, 7, 2, 3)        # patch matrix, smaller: sits on the first call's leftovers
    _compare(big, 8, 1, part=False)
    _compare(small, 2, 2, part=True)
    _compare(big, 8, 3, part=True)


def test_result_is_the_oracles_convolution_and_no_device_memory_is_taken():
    """Full-bit and part-bit (Eq. 9) results of the allocation-free call against the oracle's direct convolution
    (accumulators bit-exact, fp32 output equal), with the driver's free-memory figure read around the second call:
    the first call has looked the array's address up, so the second must leave the figure where it was."""
    L = wl.ConvLayer("c64s2", 64, 18, 18, 128, 3, 3, 2, 1)
    batch = 3
    d = wl.conv_layer_inputs(73, 5, L, batch)
    wh, _ = oracle.decompose(d["W"], d["mask"], 8, 6, True)
    desc, x, w, hi, ws, sa = _layer_tensors(L, batch, 5)
    for part in (False, True):
        ref = oracle.conv_acc(d["X"], wh if part else d["W"], L.stride, L.pad).transpose(0, 2, 3, 1)
        acc = torch.full((batch, L.Ho, L.Wo, L.Cout), -1, dtype=torch.int32, device="cuda")
        y = torch.full((batch, L.Ho, L.Wo, L.Cout), float("nan"), dtype=torch.float32, device="cuda")
        weights = hi if part else w
        nq.nq_conv_implicit_gemm_static(x, weights, desc, ws, sa, acc, y, part_bit=part, n_bits=8, h_bits=6)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        nq.nq_conv_implicit_gemm_static(x, weights, desc, ws, sa, acc, y, part_bit=part, n_bits=8, h_bits=6)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        nq.nq_device_status()
        assert free_after == free_before
        assert np.array_equal(acc.cpu().numpy(), ref)
        assert np.array_equal(y.cpu().numpy(), oracle.dequant(ref, d["w_scale"], sa, 2 if part else 0))


def test_layer_larger_than_the_built_in_array_is_refused():
    L = wl.ConvLayer("wide", 64, 112, 112, 64, 3, 3, 1, 1)
    desc = nq.nq_conv_desc(32, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    assert nq.nq_conv_workspace_bytes(desc) > nq.NQ_CONV_STATIC_SCRATCH_BYTES
    x = torch.zeros((1,), dtype=torch.int8, device="cuda")         # never read: the call must stop at the size check
    w = torch.zeros((64, 576), dtype=torch.int8, device="cuda")
    ws = torch.ones(64, device="cuda")
    y = torch.zeros((1,), device="cuda")
    with pytest.raises(nq.NqError) as e:
        nq.nq_conv_implicit_gemm_static(x, w, desc, ws, 1.0, None, y)
    assert e.value.status == 4
