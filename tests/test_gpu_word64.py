"""The paper's packed-bit tensor (64 // k fields per unsigned 64-bit word) on the GPU: conversion to and from the
library's sliced layout, bit for bit against the oracle's two packers."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _values(rows, cols, bits, seed):
    rng = wl.rng_for(92, seed)
    lim = 1 << (bits - 1)
    return rng.integers(-lim, lim, size=(rows, cols), dtype=np.int64).astype(np.int8)


def _dev_words(words_u64):
    return torch.from_numpy(words_u64.view(np.int64)).cuda()


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("rows,cols", [(3, 130), (17, 1000), (64, 256), (5, 21), (2, 4099)])
def test_word64_to_sliced_and_back(bits, rows, cols):
    v = _values(rows, cols, bits, bits * 1000 + cols)
    words = oracle.pack_word64(v, bits)
    assert words.shape[1] == nq.nq_word64_row_words(cols, bits) == oracle.word64_row_words(cols, bits)
    sliced = nq.nq_word64_to_sliced(_dev_words(words), bits, cols)
    assert np.array_equal(sliced.cpu().numpy(), oracle.pack_sliced(v, bits))
    back = nq.nq_sliced_to_word64(sliced, bits, rows, cols)
    assert np.array_equal(back.cpu().numpy().view(np.uint64), words)
    # and the fields are what the codec's own unpack reads
    assert np.array_equal(nq.nq_unpack(sliced, bits, rows, cols).cpu().numpy(), v)


def test_paper_counts_three_and_five_bit_fields():
    # twenty-one 3-bit or twelve 5-bit weights per word ("Deployment")
    assert nq.nq_word64_row_words(21, 3) == 1 and nq.nq_word64_row_words(22, 3) == 2
    assert nq.nq_word64_row_words(12, 5) == 1 and nq.nq_word64_row_words(13, 5) == 2
    assert nq.nq_word64_row_words(10, 0) == -1 and nq.nq_word64_row_words(-1, 4) == -1


def test_nested_model_arrives_in_the_paper_format():
    """INT8 nesting INT4 + 5-bit low part shipped as packed-bit tensors, converted on the device, recomposed."""
    d = wl.gemm_inputs(93, 0, 8, 300, 520)
    W, mask = d["W"], d["mask"]
    wh, wlo = oracle.decompose(W, mask, 8, 4, True)
    hi = nq.nq_word64_to_sliced(_dev_words(oracle.pack_word64(wh, 4)), 4, 520)
    lo = nq.nq_word64_to_sliced(_dev_words(oracle.pack_word64(wlo, 5)), 5, 520)
    assert np.array_equal(nq.nq_recompose(hi, lo, 300, 520, 8, 4, True).cpu().numpy(), W)


def test_empty_and_rejected():
    out = nq.nq_word64_to_sliced(torch.zeros((0, 2), dtype=torch.int64, device="cuda"), 5, 24)
    assert out.shape[0] == 0
    with pytest.raises(ValueError):
        nq.nq_word64_to_sliced(torch.zeros((4, 3), dtype=torch.int64, device="cuda"), 5, 24)
