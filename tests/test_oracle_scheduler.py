"""Pins for the scheduler oracle: the paper's VBS constants, two hand-worked groups,
edge cases and invariants over random groups.  No GPU."""
import json
import os

import numpy as np
import pytest

from oracle import scheduler as osch
from paper_2305_13144_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def _cfg(d):
    return osch.SchedCfg(**d)


def test_vbs_table_from_paper_constants():
    g = _gold("vbs_table.json")
    cfg = osch.SchedCfg(use_vbs=True, vbs_len_threshold=g["threshold"], vbs_token_budget=g["token_budget"],
                        base_batch=g["base_batch"], min_batch=g["min_batch"], max_batch=g["max_batch"])
    for L, b in g["table"].items():
        assert osch.vbs_batch(int(L), cfg) == b, L


def test_round_pow2_linear_distance_tie_goes_down():
    assert osch.round_pow2(12800, 150) == 64          # 85.3 -> 64 (21.3 away) not 128 (42.7 away)
    assert osch.round_pow2(12800, 250) == 64          # 51.2
    assert osch.round_pow2(3, 1) == 2                 # tie between 2 and 4
    assert osch.round_pow2(6, 1) == 4                 # tie between 4 and 8
    assert osch.round_pow2(7, 1) == 8
    assert osch.round_pow2(1, 1) == 1
    assert osch.round_pow2(1, 3) == 1                 # below one clamps to one


def test_binning_rounds_up_and_keeps_exact_multiples():
    cfg = osch.SchedCfg(bin_size=50, max_new_tokens=512)
    assert [osch.bin_of(x, cfg) for x in (1, 49, 50, 51, 100, 101, 0, -7)] == [50, 50, 50, 100, 100, 150, 50, 50]
    assert osch.bin_of(9999, cfg) == 550               # clamp to max_new (512) first, then its cell
    assert osch.bin_of(37, osch.SchedCfg(bin_size=1)) == 37


def test_hand_worked_example_a():
    g = _gold("sched_example_a.json")
    cfg = _cfg(g["cfg"])
    assert [osch.bin_of(p, cfg) for p in g["pred_len"]] == g["bins"]
    r = osch.simulate(g["prompt_len"], g["pred_len"], g["true_len"], cfg)
    assert r["order"] == g["order"]
    assert len(r["batches"]) == len(g["batches"])
    for got, exp in zip(r["batches"], g["batches"]):
        assert got.rows == exp["rows"] and got.cap == exp["cap"]
        assert got.is_recompute == exp["is_recompute"]
        assert got.steps == exp["steps"] and got.failed == exp["failed"]
    assert r["steps"] == g["steps"] and r["row_steps"] == g["row_steps"]
    assert r["useful_tokens"] == g["useful_tokens"] and r["failure_ratio"] == g["failure_ratio"]
    # the reported statistics, from the hand-worked totals: 1 - 885/2220 of the row-steps are wasted; three
    # batches ran 710 steps; their ten rows sat through 2220 row-steps
    for key in ("redundancy", "avg_len", "avg_len_weighted"):
        num, den = g[key + "_num_den"]
        assert r[key] == pytest.approx(num / den, rel=1e-12), key
    # the vanilla arm in index order
    v = g["vanilla_index_order"]
    vc = _cfg({**g["cfg"], "vanilla": True})
    rv = osch.simulate(g["prompt_len"], g["pred_len"], g["true_len"], vc, perm=list(range(8)))
    assert [(b.rows, b.steps) for b in rv["batches"]] == [(b["rows"], b["steps"]) for b in v["batches"]]
    assert rv["steps"] == v["steps"] and rv["row_steps"] == v["row_steps"] and rv["failures"] == []


def test_hand_worked_example_b_vbs():
    g = _gold("sched_example_b.json")
    cfg = _cfg(g["cfg"])
    pred = []
    for count, L in g["groups"]:
        pred += [L] * count
    order, batches = osch.plan([g["prompt_len"]] * len(pred), pred, cfg)
    assert order == list(range(len(pred)))
    assert [[len(b.rows), b.cap] for b in batches] == g["batches"]


def test_cap_boundary_success_and_failure():
    cfg = osch.SchedCfg(bin_size=50, base_batch=2, max_new_tokens=512)
    r = osch.simulate([5, 5], [50, 50], [50, 51], cfg)
    assert r["failures"] == [1]
    assert r["batches"][0].steps == 50
    assert r["batches"][1].rows == [1] and r["batches"][1].steps == 51 and r["batches"][1].cap == 512


def test_small_and_ragged_groups():
    cfg = osch.SchedCfg(bin_size=50, base_batch=16)
    _, b = osch.plan([3] * 5, [10, 20, 30, 40, 45], cfg)
    assert len(b) == 1 and b[0].rows == [0, 1, 2, 3, 4] and b[0].cap == 50
    _, b = osch.plan([3] * 35, [60] * 35, cfg)
    assert [len(x.rows) for x in b] == [16, 16, 3]
    _, b = osch.plan([], [], cfg)
    assert b == []


def test_every_row_fails_then_recomputes():
    cfg = osch.SchedCfg(bin_size=50, base_batch=4, max_new_tokens=512)
    r = osch.simulate([1] * 6, [10] * 6, [200] * 6, cfg)
    assert r["failures"] == [0, 1, 2, 3, 4, 5] and r["failure_ratio"] == 1.0
    assert [(b.rows, b.cap, b.is_recompute, b.steps) for b in r["batches"]] == [
        ([0, 1, 2, 3], 50, False, 50), ([4, 5], 50, False, 50),
        ([0, 1, 2, 3], 512, True, 200), ([4, 5], 512, True, 200)]


def test_switches_fcr_off_and_no_binning():
    cfg = osch.SchedCfg(bin_size=1, base_batch=2, use_fcr=False, max_new_tokens=64)
    r = osch.simulate([1] * 4, [9, 3, 7, 5], [60, 2, 7, 5], cfg)
    assert r["order"] == [1, 3, 2, 0]
    assert all(b.cap == 64 for b in r["batches"]) and r["failures"] == []
    cfg2 = osch.SchedCfg(bin_size=1, base_batch=2, use_fcr=True, max_new_tokens=64)
    r2 = osch.simulate([1] * 4, [9, 3, 7, 5], [60, 2, 7, 5], cfg2)
    assert [b.cap for b in r2["batches"]] == [5, 9, 64] and r2["failures"] == [0]


def test_cap_equal_to_max_new_is_never_a_failure():
    cfg = osch.SchedCfg(bin_size=16, base_batch=2, max_new_tokens=64)
    r = osch.simulate([1, 1], [64, 64], [64, 64], cfg)
    assert r["failures"] == [] and r["batches"][0].cap == 64


def test_kv_budget_limits_batch():
    cfg = osch.SchedCfg(bin_size=50, base_batch=16, use_vbs=True, max_new_tokens=512,
                        kv_budget_bytes=1000 * 10, kv_bytes_per_token=10)
    # each row worst case 100 + 50 = 150 tokens -> 6 rows fit in 1000 tokens
    _, b = osch.plan([100] * 20, [50] * 20, cfg)
    assert [len(x.rows) for x in b] == [6, 6, 6, 2]
    # a single row always forms a batch, even over budget
    _, b = osch.plan([5000], [50], cfg)
    assert [len(x.rows) for x in b] == [1]


@pytest.mark.parametrize("seed", range(6))
def test_invariants_random_groups(seed):
    rng = np.random.default_rng(seed)
    g = synth.make_group(257, vocab=100, eos_id=2, prompt_lo=4, prompt_hi=60, resp="lognormal",
                         max_new=512, noise_sigma=40.0, seed=seed)
    cfg = osch.SchedCfg(bin_size=int(rng.choice([1, 16, 50])), base_batch=int(rng.choice([4, 16])),
                        use_vbs=bool(seed % 2), use_fcr=bool((seed // 2) % 2 == 0), max_new_tokens=512,
                        kv_budget_bytes=int(rng.choice([0, 40000])) * 8, kv_bytes_per_token=8)
    r = osch.simulate(g.prompt_len, g.pred_len, g.true_len, cfg)
    first = [b for b in r["batches"] if not b.is_recompute]
    rec = [b for b in r["batches"] if b.is_recompute]
    assert sorted(x for b in first for x in b.rows) == list(range(g.n))
    assert [x for b in first for x in b.rows] == r["order"]
    assert [x for b in rec for x in b.rows] == r["failures"]
    assert len(set(r["failures"])) == len(r["failures"])
    for b in first:
        longest = max(osch.bin_of(g.pred_len[x], cfg) for x in b.rows)
        assert len(b.rows) <= osch.vbs_batch(longest, cfg)
        if cfg.kv_budget_bytes and len(b.rows) > 1:
            worst = max(g.prompt_len[x] for x in b.rows) + min(longest, cfg.max_new_tokens)
            assert len(b.rows) * worst * cfg.kv_bytes_per_token <= cfg.kv_budget_bytes
        for x in b.rows:
            assert (x in b.failed) == (g.true_len[x] > b.cap and b.cap < cfg.max_new_tokens)
    if not cfg.use_fcr:
        assert r["failures"] == []
    assert r["useful_tokens"] == int(g.true_len.sum())
    assert 0.0 <= r["redundancy"] < 1.0
    # a perfect predictor never fails
    r2 = osch.simulate(g.prompt_len, g.true_len, g.true_len, cfg)
    assert r2["failures"] == []


def test_vanilla_batches_are_permutation_chunks():
    g = synth.group_tiny(seed=3)
    perm = synth.make_permutation(g.n, seed=9)
    cfg = osch.SchedCfg(base_batch=8, max_new_tokens=64, vanilla=True)
    r = osch.simulate(g.prompt_len, g.pred_len, g.true_len, cfg, perm=perm)
    assert r["order"] == perm.tolist()
    assert [b.rows for b in r["batches"]] == [perm[i:i + 8].tolist() for i in range(0, 32, 8)]
    assert all(b.cap == 64 and not b.is_recompute for b in r["batches"])
    assert [b.steps for b in r["batches"]] == [int(g.true_len[perm[i:i + 8]].max()) for i in range(0, 32, 8)]


def test_scheduling_beats_vanilla_on_the_large_synthetic_group():
    """Sanity band only (dataset dependent in the paper: 66% -> 33% redundant tokens)."""
    g = synth.group_7b_1024(seed=0)
    van = osch.simulate(g.prompt_len, g.pred_len, g.true_len,
                        osch.SchedCfg(vanilla=True), perm=synth.make_permutation(g.n, 0))
    sch = osch.simulate(g.prompt_len, g.pred_len, g.true_len, osch.SchedCfg())
    assert 0.5 < van["redundancy"] < 0.75
    assert sch["redundancy"] < van["redundancy"] - 0.15
    assert sch["steps"] < van["steps"]
