"""Sampled decoding on the GPU (ss_set_sampling) against the sampling oracle, through the C ABI.

Teacher-forced: the oracle generates every row at temperature 0.5 with its counter-based draws, the engine
is forced onto the oracle's tokens, and at every step the engine's OWN draw (ss_step_opts.dump_choice) is
compared with the oracle's.  Both sides draw the same Gumbel noise from the same counters, so the tokens must
be identical wherever the oracle's decision is clear: where its best and second-best perturbed values
(logit / T + noise) are closer than twice the logit tolerance divided by T, the engine's bf16 logits may
legitimately tip the draw, and such steps are only required to pick one of the two."""
import numpy as np
import pytest

from oracle import decoder as od
from oracle import sampler as smp
from paper_2305_13144_b200 import synth
from parity_util import LOGIT_TOL, engine, oracle_model

pytestmark = pytest.mark.gpu


def test_sampled_choices_match_oracle_draws_teacher_forced():
    import torch
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    model = oracle_model(shape, w)
    g = synth.group_tiny(seed=4)
    B, cap, T, seed = 12, 20, 0.5, (7 << 32) + 12345
    keys = [100 + 3 * r for r in range(B)]                 # not 0..B-1: the row key is an input
    prompts = [g.prompt(i).tolist() for i in range(B)]
    targets = [int(min(g.true_len[i], cap + 5)) for i in range(B)]
    ref = [od.generate(model, prompts[r], cap, targets[r], keep_logits=True, temperature=T, seed=seed, row_key=keys[r])
           for r in range(B)]
    greedy = [od.generate(model, prompts[r], cap, targets[r])["tokens"] for r in range(B)]
    assert sum(a["tokens"] != b for a, b in zip(ref, greedy)) >= B // 2          # the draws do change the text
    eng = engine(shape, w, max_batch=16, max_ctx=128, max_new=32)
    api.ss_set_sampling(eng, T, seed)
    api.ss_set_row_keys(eng, keys)
    toks = np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts])
    cu = np.zeros(B + 1, dtype=np.int32)
    cu[1:] = np.cumsum([len(p) for p in prompts])
    dl = torch.zeros(B, shape.vocab, dtype=torch.float32, device="cuda")
    ch = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    steps = max(len(r["tokens"]) for r in ref)
    clear = unclear = 0
    for t in range(steps):
        forced = torch.tensor([ref[r]["tokens"][t] if len(ref[r]["tokens"]) > t else shape.eos_id for r in range(B)],
                              dtype=torch.int32, device="cuda")
        if t == 0:
            api.ss_prefill(eng, toks, cu, np.asarray(targets, dtype=np.int32), cap, forced_tokens=forced,
                           dump_logits=dl, dump_choice=ch)
        else:
            api.ss_decode_step(eng, forced_tokens=forced, dump_logits=dl, dump_choice=ch)
        torch.cuda.synchronize()
        got = ch.cpu().numpy()
        for r in range(B):
            if len(ref[r]["tokens"]) <= t or t + 1 == targets[r]:
                continue                                   # finished, or the step whose token is the forced EOS
            lg = ref[r]["logits"][t]
            z = smp.perturbed(lg, T, seed, keys[r], t + 1)
            z[shape.eos_id] = -np.inf                      # forced-length rows never draw EOS
            order = np.argsort(-z, kind="stable")
            assert order[0] == ref[r]["tokens"][t]
            if z[order[0]] - z[order[1]] > 2 * LOGIT_TOL * np.max(np.abs(lg)) / T:
                assert got[r] == order[0], (t, r)
                clear += 1
            else:
                assert got[r] in (order[0], order[1]), (t, r)
                unclear += 1
    assert clear > 100 and clear > 5 * unclear, (clear, unclear)
    api.ss_read_batch(eng, B, cap)
    api.ss_release_batch(eng)
    api.ss_set_sampling(eng, 0.0, 0)


def test_sampled_group_repeats_for_a_seed_differs_between_seeds_and_survives_recomputation():
    """Free-running through ss_run_group(): the same seed gives the same tokens twice; another seed gives other
    tokens; and because a draw depends only on (seed, query, token index, logits), the rows that FCR cuts and
    regenerates from the prompt end with exactly the tokens they have in a run without FCR."""
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    eng = engine(shape, w, max_batch=16, max_ctx=128, max_new=64, kv_tokens=16 * 128)
    g = synth.group_tiny(seed=1)
    runs = {}
    for name, seed, fcr in (("a", 5, True), ("b", 5, True), ("c", 6, True), ("nofcr", 5, False)):
        api.ss_set_sampling(eng, 0.5, seed)
        cfg = api.sched_cfg(bin_size=16, base_batch=8, max_new_tokens=64, use_fcr=fcr)
        runs[name] = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, None, g.true_len)
    api.ss_set_sampling(eng, 0.0, 0)
    cfg = api.sched_cfg(bin_size=16, base_batch=8, max_new_tokens=64)
    greedy = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, None, g.true_len)
    assert (runs["a"]["tokens"] == runs["b"]["tokens"]).all()
    assert (runs["a"]["tokens"] != runs["c"]["tokens"]).any()
    assert (runs["a"]["tokens"] != greedy["tokens"]).any()
    assert runs["a"]["stats"]["n_failed"] > 0
    assert (runs["a"]["tokens"] == runs["nofcr"]["tokens"]).all()
    for r in runs.values():
        assert r["len"].tolist() == g.true_len.tolist()
