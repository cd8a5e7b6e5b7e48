"""K2 + K4 parity: decode through the C ABI against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from helpers import OracleView, assert_close
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run_decode(w, policy=None, source="device", layer=0, deferred=False):
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    pa = PathAttention(w, layers=1, policy=policy)
    pa.write_nodes(source)
    pa.build()
    if deferred:  # the form the benchmark times: nothing waits for the host between build and decode
        pa.build(deferred=True)
    q = pa.make_q(layer, source)
    lse = pa.guarded(w.num_requests * w.num_q_heads * 4, "lse").view(torch.float32).view(w.num_requests, w.num_q_heads)
    out = pa.decode(layer, q, lse=lse)   # the output buffer it allocates sits between canaries too
    assert pa.status() == 0
    res = tensor_to_f64(out), tensor_to_f64(lse)
    pa.close()                           # checks the canaries around pool, workspace, out and lse
    return res


def test_device_generator_matches_host_bits():
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(0)
    pa = PathAttention(w, layers=1)
    q_dev = pa.make_q(0, "device").view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(q_dev, w.q_bits(0))
    pa.close()


@pytest.mark.parametrize("source", ["device", "host"])
def test_config0_full(source):
    w = W.make_config(0)
    out, lse = _run_decode(w, source=source)
    ref_o, ref_l = OracleView(w).decode()
    assert_close(out, ref_o, "cfg0 out")
    assert np.abs(lse - ref_l).max() < 2e-3


@pytest.mark.parametrize("policy", [None, (64, 1, 1, 1), (64, 3, 1, 2), (128, 16, 16, 4), (1024, 7, 2, 16)])
def test_config1_shape_reduced_all_requests(policy):
    w = W.make_config(1, n_requests=40, n_nodes=64, root_len=333, len_lo=1, len_hi=200, suffix_max=70)
    out, lse = _run_decode(w, policy=policy)
    ref_o, ref_l = OracleView(w).decode()
    assert_close(out, ref_o, f"cfg1-reduced policy={policy}")
    assert np.abs(lse - ref_l).max() < 2e-3


@pytest.mark.parametrize("deferred", [False, True])
def test_config1_full_size_sampled_requests(deferred):
    w = W.make_config(1)
    out, lse = _run_decode(w, deferred=deferred)
    reqs = np.random.default_rng(11).choice(w.num_requests, size=24, replace=False).tolist()
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref_o, "cfg1 sampled")
    assert np.abs(lse[reqs] - ref_l).max() < 2e-3
    assert np.all(np.isfinite(out))


def test_config3_reduced_high_sharing():
    # every request shares the root: group sizes 1..96 exercise ragged request tiles
    w = W.make_config(3, n_requests=96, n_nodes=64, root_len=1500, len_lo=5, len_hi=130, suffix_max=40)
    out, _ = _run_decode(w)
    ref_o, _ = OracleView(w).decode()
    assert_close(out, ref_o, "cfg3-reduced")


def test_config4_shape_reduced_with_empty_nodes():
    w = W.make_config(4, layers=1, n_requests=64, n_nodes=300, token_budget=20000, suffix_max=100)
    out, _ = _run_decode(w)
    ref_o, _ = OracleView(w).decode()
    assert_close(out, ref_o, "cfg4-reduced")


@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 64), (8, 2, 64), (4, 1, 128), (8, 8, 128), (16, 2, 128)])
def test_head_shapes(hq, hkv, d):
    w = W.make_config(0, hq=hq, hkv=hkv, d=d, n_requests=19, root_len=77, len_lo=1, len_hi=90)
    out, _ = _run_decode(w)
    ref_o, _ = OracleView(w).decode()
    assert_close(out, ref_o, f"heads {hq}/{hkv}/{d}")


def test_single_request_single_token_and_split_invariance():
    # one request, one node, one token: softmax over a single key returns its value row
    w = W.make_config(0, n_requests=1, n_nodes=2, root_len=1, depth_lo=1, depth_hi=2, suffix_max=0, len_lo=1, len_hi=1)
    w.path_ptr = np.array([0, 1], dtype=np.int32)
    w.path_node = np.array([0], dtype=np.int32)
    out, lse = _run_decode(w, source="host")
    _, v = w.node_kv_bits(0, 0)
    assert np.array_equal(out[0], W.bf16_bits_to_f64(v)[0])
    # chunking a segment differently must not change the result beyond rounding
    w = W.make_config(1, n_requests=24, n_nodes=32, root_len=900, len_lo=100, len_hi=400, suffix_max=50)
    a, _ = _run_decode(w, policy=(64, 16, 1, 1))
    b, _ = _run_decode(w, policy=(1024, 4, 1, 16))
    assert np.abs(a - b).max() < 8e-3


def test_config3_full_size_sampled_requests():
    # 1024 requests over one 8192-token root: the launch configuration the benchmark times
    w = W.make_config(3)
    out, lse = _run_decode(w, deferred=True)
    reqs = np.random.default_rng(13).choice(w.num_requests, size=20, replace=False).tolist()
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref_o, "cfg3 sampled")
    assert np.abs(lse[reqs] - ref_l).max() < 2e-3
    assert np.all(np.isfinite(out))


def test_config4_full_size_two_layers_sampled_requests():
    # full-depth shape (2048 requests, 4096 nodes, empty control nodes), two of its layers in HBM
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(4)
    pa = PathAttention(w, layers=2)
    pa.write_nodes("device")
    pa.build()
    reqs = np.random.default_rng(17).choice(w.num_requests, size=12, replace=False).tolist()
    for layer in (0, 1):
        q = pa.make_q(layer)
        out = tensor_to_f64(pa.decode(layer, q))
        assert pa.status() == 0
        assert np.all(np.isfinite(out))
        ref_o, _ = OracleView(w, layer=layer).decode(reqs)
        assert_close(out[reqs], ref_o, f"cfg4 layer {layer} sampled")
    pa.close()


def test_wide_chunks_head_dim_64_and_single_head_groups():
    # 700 requests over 8 shared nodes: every segment is shared by >= 64 requests, so the chunks run on
    # the tensor-memory decode kernel; head_dim 64 and one query head per KV head (128 requests per tile)
    w = W.make_config(0, hq=8, hkv=8, d=64, n_requests=700, n_nodes=8, root_len=300, len_lo=70, len_hi=260,
                      depth_lo=3, depth_hi=4, suffix_max=20)
    out, lse = _run_decode(w)
    reqs = np.random.default_rng(23).choice(w.num_requests, size=40, replace=False).tolist()
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref_o, "wide d64")
    assert np.abs(lse[reqs] - ref_l).max() < 2e-3
    assert np.all(np.isfinite(out))


def test_wide_chunks_gqa4_ragged_groups():
    # groups of 65..420 requests: units with a full tile pair, a partial second tile and a single tile
    w = W.make_config(1, n_requests=420, n_nodes=12, root_len=700, len_lo=65, len_hi=400, depth_lo=3, depth_hi=4,
                      suffix_max=30)
    out, lse = _run_decode(w)
    reqs = np.random.default_rng(29).choice(w.num_requests, size=24, replace=False).tolist()
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref_o, "wide gqa4")
    assert np.abs(lse[reqs] - ref_l).max() < 2e-3


def test_request_with_an_empty_context():
    # request 0's path is one private node that holds no tokens: out = 0 and lse = -inf
    w = W.make_config(0, n_requests=6)
    lone = w.num_shared_nodes  # request 0's private node id
    w.node_len = w.node_len.copy()
    w.node_len[lone] = 0
    rest = w.path_node[w.path_ptr[1]:]
    w.path_node = np.concatenate([[lone], rest]).astype(np.int32)
    w.path_ptr = np.concatenate([[0], w.path_ptr[1:] - w.path_ptr[1] + 1]).astype(np.int32)
    out, lse = _run_decode(w, source="host")
    assert np.all(out[0] == 0.0) and np.all(np.isneginf(lse[0]))
    ref_o, _ = OracleView(w).decode(list(range(1, w.num_requests)))
    assert_close(out[1:], ref_o, "others next to an empty request")


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_small_workloads_and_policies(seed):
    """Seeded random shapes (requests, nodes, segment lengths, suffixes) and chunking policies: tables bit
    for bit and every output element against the oracle, sync and deferred builds mixed."""
    from helpers import assert_tables_equal, oracle_tables
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    rng = np.random.default_rng(seed)
    policies = [None, (64, 1, 1, 1), (64, 3, 1, 2), (128, 16, 16, 4), (1024, 7, 2, 16), (512, 16, 2, 16)]
    for _ in range(6):
        over = dict(n_requests=int(rng.integers(1, 90)), n_nodes=int(rng.integers(8, 80)), root_len=int(rng.integers(1, 700)),
                    len_lo=1, len_hi=int(rng.integers(2, 300)), suffix_max=int(rng.integers(0, 90)))
        pol = policies[int(rng.integers(0, len(policies)))]
        w = W.make_config(1, seed=int(rng.integers(1, 1 << 30)), **over)
        pa = PathAttention(w, layers=1, policy=pol)
        pa.write_nodes("device")
        pa.build()
        if rng.random() < 0.5:
            pa.build(deferred=True)
        assert_tables_equal(B.gf_tables_export(pa.tables), oracle_tables(w, policy=pol))
        out = tensor_to_f64(pa.decode(0, pa.make_q(0)))
        assert pa.status() == 0
        ref, _ = OracleView(w).decode()
        assert_close(out, ref, f"random workload {over} policy {pol}")
        pa.close()


def test_wide_chunks_eight_query_heads_per_kv_head():
    # GQA group size 8: a unit of the tensor-memory kernel is 32 requests (256 stacked rows)
    w = W.make_config(1, hq=16, hkv=2, d=128, n_requests=300, n_nodes=10, root_len=400, len_lo=65, len_hi=300,
                      depth_lo=3, depth_hi=4, suffix_max=20)
    out, lse = _run_decode(w)
    reqs = np.random.default_rng(31).choice(w.num_requests, size=24, replace=False).tolist() + [0, 31, 32, 299]
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref_o, "wide gqa8")
    assert np.abs(lse[reqs] - ref_l).max() < 2e-3
    assert np.all(np.isfinite(out))
