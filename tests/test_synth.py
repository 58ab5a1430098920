"""The seeded input generators: determinism, value structure and the shapes of the workloads."""
import numpy as np
import torch

from workloads import synth
from oracle import specext_oracle as orc


def test_std_normal_statistics_and_counter_property():
    key = synth.stream_key(1, 2, 3)
    x = synth.std_normal(key, 0, 1 << 18, "cpu")
    assert abs(float(x.mean())) < 0.01 and abs(float(x.std()) - 1.0) < 0.01
    y = synth.std_normal(key, 1000, 50, "cpu")
    assert torch.equal(x[1000:1050], y)                       # element i depends on (key, i) only
    assert not torch.equal(synth.std_normal(synth.stream_key(1, 2, 4), 0, 50, "cpu"), x[:50])


def test_trees_are_valid_and_shaped():
    for name, w in synth.WORKLOADS.items():
        parent = synth.make_tree(w)
        assert parent.shape == (w.n_tree,) and parent.dtype == np.int32
        orc.ancestor_mask(parent)                              # raises on an invalid tree
        if w.tree == "levels":
            dep = orc.depth(parent)
            assert dep.max() == 5 and np.all(dep == np.arange(60) // 10)
    assert np.array_equal(synth.make_tree(synth.WORKLOADS["c1"]), synth.make_tree(synth.WORKLOADS["c1"]))


def test_layer_shapes_and_growth_property():
    w = synth.WORKLOADS["c0"]
    t = synth.make_layer(w)
    assert t["Q"].shape == (8, 4, 64) and t["K_prefix"].shape == (1024, 1, 64)
    assert t["Q"].dtype == torch.bfloat16
    w3 = synth.WORKLOADS["c3"]
    a = synth.make_layer(w3.with_prefix(1024), capacity=2048)
    b = synth.make_layer(w3.with_prefix(2048), capacity=4096)
    assert torch.equal(a["K_prefix"][:2048], b["K_prefix"][:2048])   # position j depends on (seed, j) only
    assert torch.equal(a["V_prefix"][:2048], b["V_prefix"][:2048])
    l0 = synth.make_layer(synth.WORKLOADS["c1"].with_prefix(256), layer=0)
    l1 = synth.make_layer(synth.WORKLOADS["c1"].with_prefix(256), layer=1)
    assert not torch.equal(l0["K_prefix"], l1["K_prefix"])


def test_needles_take_most_of_the_mass():
    w = synth.WORKLOADS["c1"].with_prefix(2048)
    t = synth.make_layer(w, background="graded")
    parent = synth.make_tree(w)
    f = lambda x: x.double().numpy()
    _, _, cs = orc.verify_attn(f(t["Q"]), f(t["K_prefix"]), f(t["V_prefix"]), f(t["K_tree"]),
                               f(t["V_tree"]), parent, w.chunk_size)
    _, needles = synth.needle_profile(w, w.n_chunks, "graded")
    idx = orc.select_chunks(cs[37].astype(np.float32), w.prefix_len, w.chunk_size, 8)
    assert set(needles.tolist()) <= set(idx.tolist())
    assert cs[37][needles].sum() > 0.5
