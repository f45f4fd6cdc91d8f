"""Failure detection on the GPU without a fault: a bounded wait that runs out must surface as
SS_ERR_DEVICE_TIMEOUT and leave the context usable.  The wait that runs out belongs to a small self-test
kernel (every SM waits at most a millisecond for an arrival that never comes; nothing else is in flight), not
to the decode kernel; nothing here traps, faults or hangs."""
import numpy as np
import pytest

from paper_2305_13144_b200 import synth
from parity_util import HIDDEN_TOL, LOGIT_TOL, engine, teacher_forced

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_and_the_context_recovers():
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    eng = engine(shape, w)
    g = synth.group_tiny(seed=0)
    prompts = [g.prompt(i).tolist() for i in range(4)]
    # an ordinary batch first, so that the barrier counter is not at its initial value
    el, eh, _ = teacher_forced(shape, w, prompts, [3, 2, 4, 3], 4, eng)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL
    assert api.ss_selftest_wait_timeout(eng, 1000) == api.SS_ERR_DEVICE_TIMEOUT
    assert api.ss_last_device_status(eng) == 0                 # reported once, then cleared
    # the next ordinary batch on the same context is still right (counter and status were reset)
    el, eh, _ = teacher_forced(shape, w, prompts, [3, 2, 4, 3], 4, eng)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL
    assert api.ss_selftest_wait_timeout(eng, 200) == api.SS_ERR_DEVICE_TIMEOUT      # and again
    res = api.ss_run_group(eng, api.sched_cfg(bin_size=16, base_batch=8, max_new_tokens=64),
                           g.prompt_tokens, g.prompt_off, g.pred_len, None, g.true_len)
    assert res["len"].tolist() == g.true_len.tolist()


def test_selftest_is_refused_while_a_batch_is_in_flight_and_limits_are_checked():
    from paper_2305_13144_b200 import api
    shape = synth.TINY.with_layers(1)
    w = synth.make_weights(shape, seed=2)
    eng = engine(shape, w)
    with pytest.raises(api.SSError):
        api.ss_set_wait_limit_ms(eng, 0)
    api.ss_set_wait_limit_ms(eng, 500)
    assert api.ss_selftest_wait_timeout(eng, 0) == api.SS_ERR_ARG
    api.ss_prefill(eng, np.arange(3, 13, dtype=np.int32), [0, 10], None, 4)
    assert api.ss_selftest_wait_timeout(eng, 100) == api.SS_ERR_STATE
    api.ss_decode_step(eng)                                     # with the shorter limit in force, still fine
    _, lens, _ = api.ss_read_batch(eng, 1, 4)
    assert lens[0] == 2
    api.ss_release_batch(eng)
