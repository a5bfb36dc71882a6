"""The layer tables and generators that stand in for the paper's ImageNet models."""
import numpy as np

from paper_2506_17870_b200 import workloads as wl


def test_resnet18_table_matches_the_papers_weight_count():
    L = wl.resnet18_layers()
    assert len(L) == 21
    # the similarity analysis concatenates 11,157,504 ResNet-18 weights: every convolution except
    # the 7x7 stem and the classifier
    nested = sum(l.weights for l in L if l.name not in ("conv1", "fc"))
    assert nested == 11_157_504
    assert sum(l.weights for l in L) == 11_678_912
    views = [l.gemm_view(32) for l in L]
    assert views[0] == (401408, 64, 147) and views[-1] == (32, 1000, 512)
    assert (1568, 512, 4608) in views and (25088, 128, 64) in views


def test_resnet101_and_vit_tables():
    L = wl.resnet101_layers()
    assert len(L) == 105
    assert sum(l.weights for l in L) == 44_442_816
    assert max(l.gemm_view(128)[0] for l in L) == 1_605_632
    V = wl.vit_b16_linears()
    assert len(V) == 48 and sum(k * n for _, k, n in V) == 84_934_656


def test_generators_are_seeded_and_in_range():
    a, b = wl.config1(), wl.config1()
    for k in ("W", "X", "mask", "w_scale"):
        assert np.array_equal(a[k], b[k])
    assert a["W"].dtype == np.int8 and a["mask"].dtype == np.uint8 and set(np.unique(a["mask"])) == {0, 1}
    assert a["w_scale"].min() >= 1e-3 and a["w_scale"].max() <= 1e-2
    assert abs(float(a["X"].astype(np.float64).std()) - 32.0) < 2.0
    w, s = wl.heavy_tail_weights_int8(wl.rng_for(5, 0), (64, 768))
    assert np.abs(w).max() == 127 and s.shape == (64,)
    lay = wl.resnet18_layers()[1]
    d = wl.conv_layer_inputs(2, 1, lay, 2)
    assert d["X"].shape == (2, 64, 56, 56) and d["X"].min() >= 0 and d["W"].shape == (64, 64, 3, 3)
    m = wl.oihw_to_ohwi_matrix(d["W"], 640)
    assert m.shape == (64, 640) and np.array_equal(m[:, :576].reshape(64, 3, 3, 64), d["W"].transpose(0, 2, 3, 1))
