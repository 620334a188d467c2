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


def test_percentiles_of_window_times():
    assert bench._percentiles([]) is None
    assert bench._percentiles([3.0]) == [3.0, 3.0, 1]
    xs = [float(i) for i in range(1, 101)]
    assert bench._percentiles(xs) == [50.0, 99.0, 100]


def test_paired_steps_read_the_cache_once():
    """With the beacon's queries riding on the token's pass, a window-fill step reads what the token
    reads and nothing more; unpaired, the beacon's pass reads the same stored entries again."""
    class R(bench._Passes):
        pass
    r = R()
    r.P, r.c, r.n = 512, 4, 64
    r.w = type("W", (), {"entry_bytes": 4096})()
    r.paired = False
    reg, bea = r.kv_bytes(8, 8)
    assert reg == sum(bench.entries_attended(512, n, 4) for n in range(9, 17)) * 4096 * 64
    assert bea == sum(bench.entries_beacon_query(512, n, 4) for n in (12, 16)) * 4096 * 64
    assert all(bench.entries_beacon_query(512, n, 4) == bench.entries_attended(512, n, 4) for n in (12, 16))
    r.paired = True
    assert r.kv_bytes(8, 8) == (reg, 0)


def test_step_kinds_when_fewer_steps_than_a_window_are_timed():
    """The timed graph holds exactly the K timed steps, whatever K is; with K < c it holds part of a
    window: no window-filling step, or exactly one."""
    assert bench.step_kinds(8160, 20, 32) == (20, 0)        # steps 8161..8180: the window fills at 8192
    assert bench.step_kinds(8180, 20, 32) == (19, 1)        # steps 8181..8200 contain 8192
    assert bench.step_kinds(8176, 20, 16) == (19, 1)        # 8177..8196: 8192
    assert bench.step_kinds(8184, 20, 8) == (18, 2)         # 8192, 8200
    assert bench.step_kinds(8182, 20, 2) == (10, 10)
    assert bench.step_kinds(8000, 20, 1) == (20, 0)         # uncompressed: never fills
    assert sum(bench.step_kinds(7936, 512, 32)) == 512 and bench.step_kinds(7936, 512, 32)[1] == 16
