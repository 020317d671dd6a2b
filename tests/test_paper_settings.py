"""The settings the paper prints (tests/golden/paper_settings.txt), against the binding's defaults
and the oracle: the thresholds are the defaults, and with the paper's window the retained counts are
window rows plus selected rows (64 = 32 + 32 for the smallest budget)."""
import os

import numpy as np
import pytest

import oracle
from paper_2507_19906_b200 import binding as cd, workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_settings.txt")


def _settings():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        name, vals = parts[0], []
        for tok in parts[1:]:
            try:
                vals.append(float(tok))
            except ValueError:
                break
        out[name] = vals
    return out


def test_thresholds_are_the_binding_defaults():
    s = _settings()
    p = cd.make_params(B=1, Hq=4, Hkv=2, L=300, window=32, pool=5, budget=64, n_cal=1, cap=64)
    assert p.theta1 == pytest.approx(s["theta1"][0]) and p.theta2 == pytest.approx(s["theta2"][0])
    assert p.theta1 < p.theta2          # the recompute threshold lies below the calibration threshold


@pytest.mark.parametrize("budget", [64, 128, 256, 512])
def test_oracle_with_the_papers_window_pool_and_budgets(budget):
    s = _settings()
    assert float(budget) in s["retained_tokens"]
    W, pool = int(s["snapkv_window"][0]), int(s["snapkv_pool"][0])
    cfg = wl.small_config(B=1, Hq=4, Hkv=2, L=1100, window=W, pool=pool, budget=budget, steps=1)
    Q = wl.gen_q_obs(cfg)
    K, V = wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=1)
    assert r.kept_idx.shape == (1, 2, budget)
    for h in range(2):
        kept = r.kept_idx[0, h]
        assert np.all(np.diff(kept) > 0)                                    # ascending, no duplicates
        np.testing.assert_array_equal(kept[budget - W:], np.arange(1100 - W, 1100))   # the window rows
        assert np.all(kept[:budget - W] < 1100 - W)                         # budget - window selected candidates
    # the decode gate at the printed thresholds: a query equal to the calibration query merges,
    # one orthogonal to it raises the recompute flag and does not merge
    q_same = np.ascontiguousarray(Q[:, :, W - 1])
    o = oracle.decode(q_same, None, None, r.K_kept.copy(), r.V_kept.copy(), budget, r.O_c, r.LSE_c, r.C_q,
                      theta1=s["theta1"][0], theta2=s["theta2"][0])
    assert np.all(o.flags & 1 == 1) and np.all(o.flags & 2 == 0)
    rng = np.random.Generator(np.random.Philox(key=[3, budget]))
    q_far = wl.f32_to_bf16_bits(rng.standard_normal(q_same.shape).astype(np.float32))
    o = oracle.decode(q_far, None, None, r.K_kept.copy(), r.V_kept.copy(), budget, r.O_c, r.LSE_c, r.C_q,
                      theta1=s["theta1"][0], theta2=s["theta2"][0])
    assert np.all(o.flags & 1 == 0) and np.all(o.flags & 2 == 2)


def test_other_baselines_settings_give_valid_kept_lists():
    """StreamingLLM with the paper's 32 sinks and H2O with its even split, at the paper's budgets."""
    s = _settings()
    n_sink, frac = int(s["streamingllm_sinks"][0]), s["h2o_local_fraction"][0]
    rng = np.random.Generator(np.random.Philox(key=[5, 5]))
    for budget in (64, 128, 256, 512):
        kept = oracle.streaming_indices(2000, budget, n_sink)
        assert kept.size == budget and np.all(np.diff(kept) > 0)
        assert np.array_equal(kept[:n_sink], np.arange(n_sink)) and kept[-1] == 1999 and kept[n_sink] == 2000 - (budget - n_sink)
        tail = int(budget * frac)
        kept = oracle.select_from_scores(rng.random(2000), tail=tail, budget=budget)
        assert kept.size == budget and np.all(np.diff(kept) > 0)
        assert np.array_equal(kept[budget - tail:], np.arange(2000 - tail, 2000)) and np.all(kept[:budget - tail] < 2000 - tail)
