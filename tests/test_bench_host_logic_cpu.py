"""Host-side logic of bench.py that needs no GPU: the oracle row samples, the FLOP count of a sample, the error
summary that goes into the JSON line (and decides the exit code), and the clock-sample window."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import attn_oracle as orc  # noqa: E402
from paper_2506_12355_b200 import inputs  # noqa: E402


def small_cfg(causal=True, dtype=inputs.DTYPE_BF16):
    return inputs.AttnConfig("C3", 3, dtype, causal, 2, 3, 200, 200, 64)


def test_row_sample_covers_every_head_and_every_tile_at_the_configured_density():
    cfg = inputs.CONFIGS["C5"]
    rows = bench.oracle_sample_rows(cfg, 2731)            # every 5th row (16384 // 2731 = 5)
    per_head = rows.reshape(cfg.B * cfg.H, -1) % cfg.Sq
    assert (np.diff(per_head, axis=1) == 5).all() and (per_head[:, -1] <= cfg.Sq - 1).all()
    tiles = np.unique(per_head[0] // 128)
    assert tiles.size == cfg.Sq // 128                    # every 128-row Q tile of a head is touched
    assert np.array_equal(rows // cfg.Sq, np.repeat(np.arange(cfg.B * cfg.H), per_head.shape[1]))
    # the budgeted sample never drops below one row per tile and never exceeds the head
    for name in inputs.CONFIGS:
        c = inputs.CONFIGS[name]
        rph = bench.oracle_rows_for_budget(c, 120.0)
        assert (c.Sq + 127) // 128 <= rph <= c.Sq


def test_sample_flops_counts_visible_keys():
    cfg = small_cfg(causal=True)
    rows = np.array([0, 1, 199, 200 + 7], dtype=np.int64)
    assert bench.sample_flops(cfg, rows) == 4.0 * cfg.D * (1 + 2 + 200 + 8)
    assert bench.sample_flops(small_cfg(causal=False), rows) == 4.0 * cfg.D * 4 * 200


def test_error_summary_and_tolerance_gate():
    cfg = small_cfg()
    q, k, v = inputs.make_config_inputs(cfg)
    orun = bench.run_oracle(cfg, q, k, v, rows_per_head=50)
    assert orun["rows"].size == cfg.B * cfg.H * 50 and orun["o_ref"].shape == (orun["rows"].size, cfg.D)
    # a "GPU result" that is the oracle rounded to bf16: inside the bars, errors of the size of bf16 rounding
    o_full, lse_full = orc.attention(*(orc.widen(inputs.bits(t), cfg.dtype) for t in (q, k, v)), cfg.scale, cfg.causal)
    o_t = torch.from_numpy(o_full).to(torch.bfloat16)
    l_t = torch.from_numpy(lse_full).to(torch.float32)
    e = bench.errors_against(cfg, o_t, l_t, orun)
    assert e["within_tolerance"] and 0 < e["max_abs_o"] <= 2.0 ** -7 * 6 and e["max_abs_lse"] < 1e-5
    assert e["rows_checked"] == orun["rows"].size and 0 < e["rms_o"] < 2.0 ** -7
    # one wrong element in a sampled row: outside the bars, and the row is named
    bad_row = int(orun["rows"][17])
    o_bad = o_t.clone()
    o_bad.view(-1, cfg.D)[bad_row, 5] += 1.0
    e = bench.errors_against(cfg, o_bad, l_t, orun)
    assert not e["within_tolerance"] and e["argmax_row"] == bad_row and e["max_abs_o"] > 0.9
    # a NaN (an unwritten, poisoned output) can never pass
    o_nan = o_t.clone()
    o_nan.view(-1, cfg.D)[bad_row, 0] = float("nan")
    assert not bench.errors_against(cfg, o_nan, l_t, orun)["within_tolerance"]
    # an LSE error alone is caught as well
    l_bad = l_t.clone()
    l_bad.view(-1)[bad_row] += 0.01
    assert not bench.errors_against(cfg, o_t, l_bad, orun)["within_tolerance"]


def test_clock_window_picks_samples_inside_the_timed_region():
    s = bench.ClockSampler(0)
    s.proc = object()            # pretend a sampler ran; only window() is under test
    s.rows = [(10.0, 1500.0, 1965.0, 900.0, ["sw_power_cap"]), (10.5, 1965.0, 1965.0, 300.0, []),
              (11.0, 1900.0, 1965.0, 500.0, []), (12.0, 345.0, 1965.0, 100.0, [])]
    w = s.window(10.4, 11.1)
    assert w["samples"] == 2 and w["sm_mhz"] == 1932.5 and w["reasons"] == [] and w["window"] == "timed region"
    w = s.window(10.1, 10.2)     # shorter than the sampling period: nearest samples, and it says so
    assert w["window"] == "nearest samples" and "sw_power_cap" in w["reasons"]
    s.rows = []
    assert s.window(0, 1)["reasons"] == ["no samples"]
