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


def test_oracle_sample_covers_the_budget_and_scales_by_the_work_model():
    """the bounded oracle sample of the CPU baseline: whole rows when they fit the budget, else the first eliminations of
    one row per core, scaled to full rows by sum m^2 (the oracle updates the m x m remaining block at every step)"""
    rows, steps = bench.oracle_sample(64, 32, 8, 10.0)
    assert (rows, steps) == (32, 64) and bench.full_row_factor(64, 64) == 1.0
    rows, steps = bench.oracle_sample(3072, 768, 16, 12.0)
    assert rows == 16 and 8 <= steps < 3072
    f = bench.full_row_factor(3072, steps)
    m = np.arange(1, 3073, dtype=np.float64)
    assert np.isclose(f, (m ** 2).sum() / (m[-steps:] ** 2).sum()) and f > 1.0
    # the sampled share of a row's work is about budget / estimated row time
    est_row = bench.ORACLE_S_PER_UPDATE * (2.0 / 3.0) * 3072 ** 3
    assert 0.5 < (1.0 / f) / (12.0 / est_row) < 2.0
    assert bench.full_row_factor(10, 1) == float((np.arange(1, 11) ** 2).sum()) / 100.0
