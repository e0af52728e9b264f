"""The byte / flop model that bench.py reports for the blocked engine (host arithmetic only)."""
import numpy as np

import bench


def test_blocked_schedule_accounts_for_every_step():
    for d, panel, ms, maxp, l2 in [(2304, 44640, 209, 64, 0), (3072, 30432, 172, 64, 27), (768, 23904, 152, 64, 0), (300, 9000, 90, 3, 0)]:
        plan = {"on_chip_below": ms, "panel_floats": panel, "max_pending": maxp, "l2_vectors": l2}
        sched = bench.blocked_schedule(plan, d, d)
        sizes = [m for m, _ in sched]
        assert sizes == sorted(sizes, reverse=True) and all(nb >= 1 for _, nb in sched)
        assert d - sum(nb for _, nb in sched) == sizes[-1] and sizes[-1] <= max(ms, 1) + maxp
        for m1, nb in sched:                     # never more pending updates than fit
            m0 = m1 + nb
            assert nb <= min(maxp, panel // bench.pending_stride(m0) + l2)
        nbytes, flops = bench.blocked_bytes_flops(plan, d)
        assert nbytes > 2.0 * d * (d + 1) and flops > 0


def test_one_update_per_pass_moves_the_triangle_every_step():
    d = 200
    plan = {"on_chip_below": 0, "panel_floats": 10 ** 9, "max_pending": 1, "l2_vectors": 0}
    nbytes, flops = bench.blocked_bytes_flops(plan, d)
    m = np.arange(1, d, dtype=np.float64)        # sizes after each of the first d - 1 steps
    assert np.isclose(nbytes, 2.0 * d * (d + 1) + float((4.0 * m * (m + 1)).sum()))
    assert np.isclose(flops, float((m * (m + 1)).sum()))
    assert bench.model_bytes_full(4) == 8 * (16 + 9 + 4 + 1)
