"""ps_profile_grid through the C ABI: row order, the paper's two table keys, and
lengths that can be regenerated from each draw's seed (timings are unpinned)."""
import numpy as np
import pytest

import paper_2507_17769_b200 as ps
from workloads import gen

pytestmark = pytest.mark.gpu


def test_grid_rows_keys_and_regenerable_lengths(tmp_path):
    chunks, decodes, ctxs, seeds = (64, 512), (8, 32), (512, 2048), 2
    csv = tmp_path / "table.csv"
    rows = ps.ps_profile_grid(ps.make_shape(32, 8, 128), chunks, decodes, ctxs, seeds, 2, 3, 3000, str(csv))
    assert len(rows) == 2 * 2 * 2 * seeds
    k = 0
    for ci, c in enumerate(chunks):
        for ni, n in enumerate(decodes):
            for mi, m in enumerate(ctxs):
                cell = (ci * len(decodes) + ni) * len(ctxs) + mi
                for s in range(seeds):
                    r = rows[k]
                    k += 1
                    assert (r.chunk, r.n_decode, r.mean_ctx, r.seed_index) == (c, n, m, s)
                    assert r.seed == 3000 + seeds * cell + s and r.token_batch == c + n
                    b = gen.config3_cell(c, n, m, int(r.seed))  # same law, same generator, same seed
                    assert r.kv_tokens == int(b.kv_len.sum()) and r.prefill_prior == int(b.prior[n])
                    assert r.decode_bytes == b.decode_bytes() and abs(r.prefill_flops - b.prefill_flops()) < 1e-3 * b.prefill_flops()
                    assert 0 < r.latency_min_us <= r.latency_us <= r.latency_max_us < 1e5
                    # the rates are the row's own work over its median latency; the fraction uses the nominal peaks here
                    sec = r.latency_us * 1e-6
                    assert abs(r.decode_TBps - r.decode_bytes / sec / 1e12) <= 1e-3 * r.decode_TBps + 1e-6
                    assert abs(r.prefill_TFLOPs - r.prefill_flops / sec / 1e12) <= 1e-3 * r.prefill_TFLOPs + 1e-6
                    want = max(r.decode_bytes / 8000e9, r.prefill_flops / 2250e12) / sec
                    assert abs(r.roofline_frac - want) <= 1e-3 * want and 0 < r.roofline_frac < 1.5
    lines = csv.read_text().strip().splitlines()
    assert lines[0].startswith("component,chunk,n_decode") and len(lines) == 1 + len(rows)
    # more KV tokens at the same decode count never makes the batch faster by much
    small = np.median([r.latency_us for r in rows if r.chunk == 64 and r.n_decode == 32 and r.mean_ctx == 512])
    large = np.median([r.latency_us for r in rows if r.chunk == 64 and r.n_decode == 32 and r.mean_ctx == 2048])
    assert large > 0.8 * small


def test_grid_with_the_kv_append_in_the_timed_region(tmp_path):
    sh = ps.make_shape(32, 8, 128)
    csv = tmp_path / "t.csv"
    plain = ps.ps_profile_grid(sh, (256,), (32,), (1024,), 2, 2, 5, 3000)
    both = ps.ps_profile_grid(sh, (256,), (32,), (1024,), 2, 2, 5, 3000, str(csv), include_kv_write=True)
    assert [(r.seed, r.kv_tokens, r.token_batch) for r in plain] == [(r.seed, r.kv_tokens, r.token_batch) for r in both]
    assert all(0 < r.latency_us < 1e5 for r in both)
    # the append adds a kernel launch to every run: it cannot make the step much faster
    assert np.median([r.latency_us for r in both]) > 0.8 * np.median([r.latency_us for r in plain])
    assert csv.read_text().splitlines()[1].startswith("attn+kv_write,256,32,1024")


def test_grid_rejects_bad_specs():
    sh = ps.make_shape(32, 8, 128)
    for args in [((), (8,), (512,), 1, 1, 1), ((64,), (8,), (1,), 1, 1, 1), ((64,), (8,), (512,), 0, 1, 1), ((0,), (0,), (512,), 1, 1, 1)]:
        with pytest.raises(ps.PsError):
            ps.ps_profile_grid(sh, *args, 3000)
