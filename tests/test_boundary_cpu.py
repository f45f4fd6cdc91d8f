"""CPU checks of the boundary: the library loads, exports what the header declares, and its
host scheduler (ss_schedule) agrees bit for bit with the scheduler oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import scheduler as osch
from paper_2305_13144_b200 import api, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "seqsched.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ss_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = api.lib()
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(L, n), n
    assert sorted(api.EXPORTS) == names


def test_struct_sizes_match_header_layout():
    assert ctypes.sizeof(api.ss_model_cfg) == 36
    assert ctypes.sizeof(api.ss_runtime_cfg) == 24
    assert ctypes.sizeof(api.ss_sched_cfg) == 56
    assert ctypes.sizeof(api.ss_batch_desc) == 16
    assert ctypes.sizeof(api.ss_batch_log) == 32
    assert ctypes.sizeof(api.ss_group_stats) == 64
    assert ctypes.sizeof(api.ss_step_opts) == 32            # four pointers: forced tokens, logits, hidden, choice


def test_strerror_and_argument_errors():
    assert api.ss_strerror(0) == "ok"
    assert "key/value" in api.ss_strerror(api.SS_ERR_KV_BUDGET)
    bad = api.sched_cfg(bin_size=0)
    with pytest.raises(api.SSError) as e:
        api.ss_schedule(bad, [1], [1])
    assert e.value.code == api.SS_ERR_ARG
    with pytest.raises(api.SSError):
        api.ss_schedule(api.sched_cfg(vanilla=True), [1, 1], [1, 1], perm=[0, 0])     # not a permutation
    m = api.model_cfg(synth.TINY)
    m.head_dim = 32
    m.n_heads = 8
    with pytest.raises(api.SSError) as e:
        api.ss_arena_bytes(m, api.runtime_cfg(8, 128, 256, 64, 1024))
    assert e.value.code == api.SS_ERR_UNSUPPORTED


def _to_oracle(cfg):
    return osch.SchedCfg(bin_size=cfg.bin_size, base_batch=cfg.base_batch, use_vbs=bool(cfg.use_vbs),
                         use_fcr=bool(cfg.use_fcr), vbs_len_threshold=cfg.vbs_len_threshold,
                         vbs_token_budget=cfg.vbs_token_budget, min_batch=cfg.min_batch, max_batch=cfg.max_batch,
                         max_new_tokens=cfg.max_new_tokens, kv_budget_bytes=cfg.kv_budget_bytes,
                         kv_bytes_per_token=cfg.kv_bytes_per_token, vanilla=bool(cfg.vanilla))


def _same_plan(cfg, g, perm=None):
    order, batches = api.ss_schedule(cfg, g.prompt_len, g.pred_len, perm)
    o_order, o_batches = osch.plan(g.prompt_len, g.pred_len, _to_oracle(cfg), perm)
    assert order.tolist() == o_order
    assert len(batches) == len(o_batches)
    for (first, n, cap, rec), ob in zip(batches, o_batches):
        assert order[first:first + n].tolist() == ob.rows and cap == ob.cap and rec == 0


KV7, KV13 = 524288, 819200


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_schedule_matches_oracle_on_the_evaluation_groups(seed):
    _same_plan(api.sched_cfg(bin_size=16, base_batch=8, max_new_tokens=64), synth.group_tiny(seed))
    g = synth.group_7b_1024(seed)
    _same_plan(api.sched_cfg(), g)
    _same_plan(api.sched_cfg(vanilla=True), g, synth.make_permutation(g.n, seed))
    _same_plan(api.sched_cfg(use_vbs=True, kv_budget_bytes=120 * 10**9, kv_bytes_per_token=KV7), g)
    g13 = synth.group_13b_512(seed)
    _same_plan(api.sched_cfg(use_vbs=True, max_new_tokens=2048, kv_budget_bytes=120 * 10**9,
                             kv_bytes_per_token=KV13), g13)


@pytest.mark.parametrize("seed", range(8))
def test_schedule_matches_oracle_random_switches(seed):
    rng = np.random.default_rng(100 + seed)
    g = synth.make_group(int(rng.integers(1, 400)), vocab=50, eos_id=2, prompt_lo=1, prompt_hi=300,
                         resp="lognormal", max_new=512, noise_sigma=60.0, seed=seed)
    cfg = api.sched_cfg(bin_size=int(rng.choice([1, 7, 50, 64])), base_batch=int(rng.choice([1, 3, 16])),
                        use_vbs=bool(rng.integers(2)), use_fcr=bool(rng.integers(2)),
                        vbs_len_threshold=int(rng.choice([100, 300])), vbs_token_budget=int(rng.choice([999, 12800])),
                        min_batch=int(rng.choice([1, 16])), max_batch=int(rng.choice([64, 256])),
                        kv_budget_bytes=int(rng.choice([0, 30000])), kv_bytes_per_token=1)
    _same_plan(cfg, g)


def test_schedule_empty_group_and_capacity():
    order, batches = api.ss_schedule(api.sched_cfg(), [], [])
    assert order.tolist() == [] and batches == []
    L = api.lib()
    cfg = api.sched_cfg(base_batch=1)
    pl = np.ones(4, dtype=np.int32)
    order = np.zeros(4, dtype=np.int32)
    b = (api.ss_batch_desc * 2)()
    nb = ctypes.c_int32(0)
    rc = L.ss_schedule(ctypes.byref(cfg), pl.ctypes.data, pl.ctypes.data, None, 4, order.ctypes.data, b, 2,
                       ctypes.byref(nb))
    assert rc == api.SS_ERR_CAPACITY and nb.value == 4
