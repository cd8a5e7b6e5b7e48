"""Pins for the pool bookkeeping oracle (extents that can be released and reused)."""
import json
import os

import numpy as np

from oracle import tables as OT

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pool_release_sequence.json")


def test_hand_worked_sequence():
    g = json.load(open(GOLDEN))
    pool = OT.PoolModel(g["capacity_tiles"])
    for step in g["steps"]:
        if step["op"] == "reserve":
            assert pool.reserve(step["node"], step["tokens"]) == step["offset"], step
        else:
            pool.release(step["node"])
    assert pool.tiles_in_use() == g["final_tiles_in_use"]


def test_without_release_it_is_the_append_only_layout():
    """No release ever: first fit degenerates to extents in first-write order, each rounded up to
    whole tiles, which is what pool_offsets states independently."""
    rng = np.random.default_rng(4)
    lens = rng.integers(0, 400, size=60)
    off, end = OT.pool_offsets(range(60), lens, 60)
    pool = OT.PoolModel(1000)
    for v in range(60):
        assert pool.reserve(v, int(lens[v])) == int(off[v])
    assert pool.high_water() * OT.TILE_TOKENS == end


def test_random_sequences_keep_the_invariants():
    """Brute force: after every operation no two live extents overlap, every extent is a run of the
    stated length, a refused request really had no free run long enough, and the chosen run is the
    first one that fits (no earlier free run of that length exists)."""
    rng = np.random.default_rng(9)
    for trial in range(20):
        cap = int(rng.integers(8, 40))
        pool = OT.PoolModel(cap)
        live = {}
        nxt = 0
        for _ in range(200):
            if live and rng.random() < 0.45:
                v = int(rng.choice(list(live)))
                pool.release(v)
                del live[v]
                continue
            n = int(rng.integers(1, 6 * 64))
            need = -(-n // 64)
            taken = np.zeros(cap, dtype=bool)
            for (a, k) in live.values():
                assert not taken[a:a + k].any()
                taken[a:a + k] = True
            runs = [i for i in range(cap - need + 1) if not taken[i:i + need].any()]
            got = pool.reserve(nxt, n)
            if not runs:
                assert got is None
            else:
                assert got == runs[0] * 64
                live[nxt] = (runs[0], need)
            nxt += 1
        assert pool.tiles_in_use() == sum(k for _, k in live.values())
