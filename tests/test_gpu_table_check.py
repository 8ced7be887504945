"""The table built from a real sweep predicts held-out batches of the same law to within a loose bound (timings are
unpinned: this checks the path sweep -> ps_table_build -> ps_table_predict, not a number)."""
import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from paper_2507_17769_b200 import sched_binding as S
from paper_2507_17769_b200.table_check import rel_errors

pytestmark = pytest.mark.gpu


def test_table_from_a_sweep_predicts_held_out_decode_heavy_batches():
    shape = ps.make_shape(32, 8, 128)
    rows = ps.ps_profile_grid(shape, (64, 256), (32, 128), (1024, 4096), 3, 2, 5, 3000)
    table = S.ps_table_build(rows)
    try:
        b, icpt, slope, slope_pf = S.ps_table_get_lines(table)
        assert b.tolist() == [96, 192, 288, 384] and (slope > 0).all()   # more KV tokens cost more time
        held = ps.ps_profile_grid(shape, (128,), (64,), (2048,), 3, 2, 5, 9000)
        err = rel_errors(table, held)
        assert np.median(np.abs(err)) < 0.5
        # admission flips from yes to no as the TPOT tightens around the predicted time
        kv, rem = np.full(63, 2048, np.int32), np.full(63, 100, np.int32)
        ok, pred, peak = S.ps_admit(table, kv, rem, 2048, 100, 0, 0, 0.0, 1e9)
        assert ok and peak == 64 * (2048 + 99)
        assert not S.ps_admit(table, kv, rem, 2048, 100, 0, 0, 0.0, pred * 0.99)[0]
        # the same sweep in the overlap form: positive slopes on both sides, held-out batches within the same bound
        overlap = S.ps_table_build_overlap(rows)
        try:
            _, base, o_s, o_q = S.ps_table_get_lines(overlap)
            assert (base == 0).all() and (o_s > 0).all() and (o_q >= 0).all() and S.ps_table_get_overlap(overlap) is not None
            assert np.median(np.abs(rel_errors(overlap, held))) < 0.5
        finally:
            S.ps_table_free(overlap)
    finally:
        S.ps_table_free(table)
