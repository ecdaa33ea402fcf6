"""The split-KV partition's specification, restated in Python (helpers.expected_plan), must visit
every (request, kv head, tile) exactly once and in order for any batch and any partition width.
The GPU tests compare the kernels' own partition with this restatement."""
import numpy as np

from helpers import covered_tiles, expected_plan


def test_partition_spec_visits_every_tile_exactly_once():
    rng = np.random.default_rng(0)
    for trial in range(30):
        B = int(rng.integers(1, 20)); Hkv = int(rng.integers(1, 9)); C = int(rng.integers(1, 700))
        lens = rng.integers(1, 3000, size=B).astype(np.int32)
        tiles = (lens.astype(np.int64) + 31) // 32
        want = [(r, h, t) for r in range(B) for h in range(Hkv) for t in range(int(tiles[r]))]
        assert covered_tiles(lens, Hkv, C) == want


def test_spans_with_many_short_pieces_get_fewer_tiles():
    """The overhead units shift work away from spans that hold many (request, kv head) pieces."""
    lens = np.array([64] * 40 + [4096] * 4, dtype=np.int32)          # 2-tile requests, then long ones
    Hkv, C = 8, 64
    total, q, starts = expected_plan(lens, Hkv, C)
    counts = []
    seen = covered_tiles(lens, Hkv, C, counts=counts)
    assert sum(counts) == len(seen) == Hkv * int(((lens + 31) // 32).sum())
    cost = 3                                                         # overhead units per (request, kv head): helpers' default
    short = [n for n, s in zip(counts, starts) if 0 <= s[0] < 36]   # spans that start and end inside the short requests
    long_ = [n for n, s in zip(counts[:-1], starts[:-1]) if s[0] >= 41]
    assert short and long_
    assert max(short) <= 2 * q // (2 + cost) + 2                     # 2 of every 2 + cost units are tiles there
    assert min(long_) >= q - cost                                    # 128 of every 128 + cost units are tiles here
