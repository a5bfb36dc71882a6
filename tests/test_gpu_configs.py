"""The remaining benchmark configurations at full size, checked against the oracle on samples.

config 3: ResNet-101-shaped stack -- whole-model page-out / page-in as ONE batched call over its 105 weight
          tensors, and convolution layers at batch 128 on sampled output pixels.
config 5: ViT-B/16-shaped linears (M = 256 x 197 tokens), INT8 nesting INT4 (4-bit w_high + 5-bit w_low),
          heavy-tailed weights, both modes, on sampled rows.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_17870_b200 as nq
from paper_2506_17870_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    torch.cuda.synchronize()
    return t.cpu().numpy()


def test_config3_whole_model_page_out_and_page_in_in_one_call():
    layers = wl.resnet101_layers()
    n, h = 8, 6
    tensors, keep = [], []
    total = 0
    for i, L in enumerate(layers):
        rng = wl.rng_for(3, i)
        w, _ = wl.gaussian_weights_int8(rng, (L.Cout, L.Cin, L.R, L.S), L.K)
        mask = wl.bernoulli_mask(rng, w.shape)
        ld = -(-L.K // 16) * 16
        w_mat = dev(wl.oihw_to_ohwi_matrix(w, ld))[:, :L.K]
        m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ld))[:, :L.K]
        hi, lo = nq.nq_decompose(w_mat, m_mat, n, h, True)
        out = torch.zeros((L.Cout, ld), dtype=torch.int8, device="cuda")[:, :L.K]
        tensors.append({"w_int": out, "packed_high": hi.clone(), "packed_low": lo})
        keep.append((w_mat, hi, w, mask))
        total += L.weights
    assert len(tensors) == 105 and total == 44_442_816
    plan = nq.nq_batch_plan(tensors)
    nq.nq_recompose_batched(plan, n, h, True)                       # page-in: one launch for the model
    for t, (w_mat, hi, _, _) in zip(tensors, keep):
        assert torch.equal(t["w_int"], w_mat)
        t["packed_high"].zero_()
    nq.nq_drop_low_batched(plan, n, h, True)                        # page-out: one launch for the model
    for t, (w_mat, hi, _, _) in zip(tensors, keep):
        assert torch.equal(t["packed_high"], hi)
    # the packed bytes themselves against the oracle, on a few tensors of different shapes
    for i in (0, 1, 2, 50, 104):
        L = layers[i]
        _, hi, w, mask = keep[i]
        wh, wlo = oracle.decompose(wl.oihw_to_ohwi_matrix(w), wl.oihw_to_ohwi_matrix(mask), n, h, True)
        assert np.array_equal(host(hi), oracle.pack_sliced(wh, h))
        assert np.array_equal(host(tensors[i]["packed_low"]), oracle.pack_sliced(wlo, n - h + 1))


def _distinct_resnet101_shapes():
    """The first layer of every distinct (Cin, H, W, Cout, R, S, stride, pad) of the stack: 24 shapes, the
    7 x 7 stem (explicit patch matrix) and the classifier included."""
    seen, names = set(), []
    for L in wl.resnet101_layers():
        key = (L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad)
        if key not in seen:
            seen.add(key)
            names.append(L.name)
    return names


@pytest.mark.parametrize("name,h", [(n, 6) for n in _distinct_resnet101_shapes()] +
                         [("l3b1c1", 4), ("l4b0c2", 4), ("l1b0c3", 3)])
def test_config3_convolution_layers_at_batch_128_sampled_pixels(name, h):
    L = next(l for l in wl.resnet101_layers() if l.name == name)
    batch = 128
    d = wl.conv_layer_inputs(3, 7, L, batch)
    X, W, mask, ws, sa = d["X"], d["W"], d["mask"], d["w_scale"], d["act_scale"]
    wh, _ = oracle.decompose(W, mask, 8, h, True)
    ldw = -(-L.K // 16) * 16
    w_mat = dev(wl.oihw_to_ohwi_matrix(W, ldw))[:, :L.K]
    m_mat = dev(wl.oihw_to_ohwi_matrix(mask, ldw))[:, :L.K]
    hi, _ = nq.nq_decompose(w_mat, m_mat, 8, h, True)
    desc = nq.nq_conv_desc(batch, L.Cin, L.H, L.W, L.Cout, L.R, L.S, L.stride, L.pad, 1)
    rng = wl.rng_for(3, 99)
    Ho, Wo = L.Ho, L.Wo
    pts = {(0, 0, 0), (batch - 1, Ho - 1, Wo - 1), (0, Ho - 1, 0), (batch - 1, 0, Wo - 1), (63, Ho // 2, Wo // 2)}
    pts |= {(int(rng.integers(batch)), int(rng.integers(Ho)), int(rng.integers(Wo))) for _ in range(30)}
    pix = np.array(sorted(pts), dtype=np.int64)
    idx = torch.from_numpy(pix).cuda()
    x_dev, wsd = dev(X), dev(ws)
    for part in (False, True):
        acc, y, _ = nq.nq_conv_implicit_gemm(x_dev, hi if part else w_mat, desc, wsd, sa, part_bit=part, n_bits=8, h_bits=h,
                                             want_acc=True, y_dtype=torch.bfloat16)
        nq.nq_device_status()
        ref = oracle.conv_acc_pixels(X, wh if part else W, L.stride, L.pad, pix)
        assert np.array_equal(host(acc[idx[:, 0], idx[:, 1], idx[:, 2]]), ref)
        y_ref = oracle.dequant(ref, ws, sa, 8 - h if part else 0)
        got = host(y[idx[:, 0], idx[:, 1], idx[:, 2]].view(torch.int16)).view(np.uint16)
        assert np.array_equal(got, oracle.f32_to_bf16_bits(y_ref))


@pytest.mark.parametrize("name,K,N", [("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768)])
def test_config5_vit_linears_int8_nesting_int4(name, K, N):
    M = 256 * wl.VIT_TOKENS
    d = wl.vit_linear_inputs({"qkv": 0, "proj": 1, "fc1": 2, "fc2": 3}[name], M, K, N)
    W, X, mask, ws, sa = d["W"], d["X"], d["mask"], d["w_scale"], d["act_scale"]
    n, h = 8, 4
    wh, wlo = oracle.decompose(W, mask, n, h, True)
    hi, lo = nq.nq_decompose(dev(W), dev(mask), n, h, True)
    assert hi.shape[1] == K // 2 and lo.shape[1] == K * 5 // 8          # 4-bit w_high, 5-bit w_low
    assert np.array_equal(host(hi), oracle.pack_sliced(wh, 4)) and np.array_equal(host(lo), oracle.pack_sliced(wlo, 5))
    w_rec = nq.nq_recompose(hi, lo, N, K, n, h, True)
    assert np.array_equal(host(w_rec), W)
    assert torch.equal(nq.nq_drop_low(w_rec, lo, n, h, True), hi)
    rng = wl.rng_for(5, 50)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 257, M - 1], rng.integers(0, M, 48)]))
    rows_t = torch.from_numpy(rows).cuda()
    Xd, wsd = dev(X), dev(ws)
    for part in (False, True):
        Wref = wh if part else W
        if part:
            acc, y = nq.nq_gemm_part(Xd, hi, N, n, h, wsd, sa, want_acc=True)
        else:
            acc, y = nq.nq_gemm_full(Xd, w_rec, wsd, sa, want_acc=True)
        nq.nq_device_status()
        ref = oracle.gemm_acc(X[rows], Wref)
        assert np.array_equal(host(acc[rows_t]), ref)
        y_ref = oracle.dequant(ref, ws, sa, 4 if part else 0)
        got = host(y[rows_t])
        assert np.max(np.abs(got - y_ref)) <= 1e-5 * np.max(np.abs(y_ref))
        assert np.array_equal(got, y_ref)
        acc64 = host(acc).astype(np.int64)
        assert np.array_equal(acc64.sum(axis=0), Wref.astype(np.int64) @ X.astype(np.int64).sum(axis=0))
