"""The synthetic input generator: determinism, value distribution, DAG and path shape."""
import numpy as np
import torch

from paper_2605_22566_b200 import workloads as W


def test_quantile_table_and_rounding():
    tab = W.quantile_table()
    assert tab.shape == (65536,) and tab.dtype == np.uint16
    x = W.bf16_bits_to_f64(tab)
    assert np.all(np.diff(x) >= 0) and np.allclose(x, -x[::-1])
    assert abs(x.mean()) < 1e-6 and abs(x.std() - 1.0) < 2e-3
    # round-to-nearest-even agrees with the library's fp32 -> bf16 conversion
    f = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    ref = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(W.f32_to_bf16_bits(f), ref)


def test_streams_are_counter_based():
    key = W.stream_key(7, W.KIND_K, 3, 11)
    a = W.fill_bits(key, 0, 1000)
    assert np.array_equal(W.fill_bits(key, 250, 100), a[250:350])
    assert not np.array_equal(W.fill_bits(W.stream_key(7, W.KIND_V, 3, 11), 0, 1000), a)
    # scalar restatement of one element
    i = 123
    h = W.mix64_int(key + (i + 1) * W.GOLDEN)
    assert a[i] == W.quantile_table()[h & 0xFFFF]
    x = W.bf16_bits_to_f64(W.fill_bits(key, 0, 1 << 18))
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01


def test_configs_have_the_stated_shape():
    for cfg in range(5):
        a, b = W.make_config(cfg), W.make_config(cfg)
        assert np.array_equal(a.path_node, b.path_node) and np.array_equal(a.node_len, b.node_len)
        edges = set(zip(a.edge_src.tolist(), a.edge_dst.tolist()))
        assert all(s < d for s, d in edges)  # ids ascend along edges: acyclic
        for r in range(a.num_requests):
            p = a.path(r).tolist()
            assert p[0] == 0 and len(set(p)) == len(p)
            shared = [v for v in p if v < a.num_shared_nodes]
            assert all((x, y) in edges for x, y in zip(shared[:-1], shared[1:]))
    w = W.make_config(1)
    assert (w.num_q_heads, w.num_kv_heads, w.head_dim, w.num_requests) == (32, 8, 128, 256)
    assert w.node_len[0] == 2048 and w.node_len[1:256].min() >= 128 and w.node_len[1:256].max() <= 1024
    depth = np.array([sum(1 for v in w.path(r) if v < 256) for r in range(256)])
    assert depth.min() >= 4 and depth.max() <= 8
    w = W.make_config(2)
    pre = w.request_len() - 512
    assert w.mode == "extend" and pre.min() >= 2048 and pre.max() <= 12288
    assert all(4 <= g <= 20 for g in w.notes["groups"]) and sum(w.notes["groups"]) == 64
    w = W.make_config(3)
    assert np.all(w.path_node[w.path_ptr[:-1]] == 0) and w.node_len[0] == 8192
    assert w.materialised_tokens() > 20 * w.resident_tokens()
    w = W.make_config(4)
    assert int(w.node_len[:4096].sum()) == 524288 and w.num_layers == 32
