"""bench.py's byte accounting against the oracle's closed forms and its literal cache (CPU)."""
import numpy as np

import bench
from oracle.breadcrumbs_oracle import SeqCache, closed_form_length


def test_entries_attended_equal_the_literal_cache_length():
    for P, c in [(5, 4), (0, 2), (17, 16), (3, 1), (8, 32)]:
        s = SeqCache(1, c)
        z = np.zeros((1, 2))
        s.prefill(0, np.zeros((P, 1, 2)), np.zeros((P, 1, 2)))
        for n in range(1, 3 * max(c, 4) + 2):
            s.append(0, z, z)
            assert bench.entries_attended(P, n, c) == len(s.cache[0])          # what the n-th token's query reads
            if c > 1 and s.window_len(0) == c:
                assert bench.entries_beacon_query(P, n, c) == len(s.cache[0])  # stored entries the beacon query reads
                s.compress(0, z, z)
            assert len(s.cache[0]) == closed_form_length(P, n, c)


def test_traffic_table_covers_the_sweep():
    assert set(bench.TRAFFIC_OVER_ALGORITHMIC) == set(bench.RATIOS)
    assert all(0.9 < v <= 1.0 for v in bench.TRAFFIC_OVER_ALGORITHMIC.values())
