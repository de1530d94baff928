"""The paper's per-window timing model against the numbers it prints (Table 4 and the text below it)."""
import pytest

from paper_2607_28144_b200 import timing_model as tm


def test_table_4_decomposition():
    t = tm.PAPER_TABLE_4
    assert t.diffusion_path() == 513.0                      # "w_d + d ~ 513 ms"
    assert t.v + t.a == 459.0 and t.w_e + t.e == 458.0      # decode and encode branches, "balanced by design"
    assert t.vae_path() == 459.0
    assert t.window_ms() == 972.0                           # "the two paths sum to ~972 ms"
    assert tm.realtime_budget_ms(24, 24.0) == 1000.0        # stride S = F - 1 = 24 frames at 24 fps
    assert tm.feasible(t) and tm.realtime_budget_ms() - t.window_ms() == pytest.approx(28.0)  # "~28 ms headroom"


def test_overlap_and_levers():
    t = tm.PAPER_TABLE_4
    assert t.serial_ms() == 78 + 435 + 399 + 60 + 301 + 157 and t.serial_ms() > 1000.0  # without overlap: infeasible
    assert not tm.feasible(tm.WindowTerms(t.w_d, t.d, t.v, t.a, t.e, t.w_e + 100.0), 1000.0)  # encode branch dominates
    eager = tm.WindowTerms(t.w_d + 33.0, t.d, t.v, t.a, t.e, t.w_e)   # torch.compile saves ~33 ms of w_d (1005 -> 972)
    assert eager.window_ms() == 1005.0 and not tm.feasible(eager)
    faster = tm.with_attention_ms(t, 200.0, 91.0)
    assert faster.window_ms() == pytest.approx(972.0 - 109.0)
