"""ss_run_group() on the GPU against the scheduler oracle, bit-exact, with every switch of Sec. 4.1 / Table 5:
variable batch size with batches of up to 256 rows, a key/value budget that cuts batches, FCR off, no binning --
and one group that ends by natural EOS (no forced lengths), where the oracle DECODER supplies the lengths.
Small model, so that a thousand-query group runs in seconds."""
import numpy as np
import pytest

from oracle import decoder as od
from oracle import scheduler as osch
from paper_2305_13144_b200 import synth
from parity_util import LOGIT_TOL, assert_group_matches_simulation, engine, oracle_model, oracle_sched_cfg

pytestmark = pytest.mark.gpu

KV_TOK_TINY = 2 * synth.TINY.d_model * 2 * synth.TINY.n_layers        # bytes of keys + values per cached token


def _group(n, seed):
    return synth.make_group(n, vocab=synth.TINY.vocab, eos_id=synth.TINY.eos_id, prompt_lo=8, prompt_hi=32,
                            resp="uniform", max_new=64, noise_sigma=8.0, seed=seed)


@pytest.fixture(scope="module")
def wide_engine():
    w = synth.make_weights(synth.TINY, seed=1234)
    return engine(synth.TINY, w, max_batch=256, max_ctx=128, max_prefill=8192, max_new=64, kv_tokens=256 * 128)


def _run_and_compare(eng, g, cfg, perm=None):
    from paper_2305_13144_b200 import api
    res = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, perm, g.true_len)
    sim = osch.simulate(g.prompt_len, g.pred_len, g.true_len, oracle_sched_cfg(cfg), perm)
    assert_group_matches_simulation(res, sim, g.n, g.true_len, synth.TINY.eos_id)
    assert api.ss_last_device_status(eng) == 0
    return res, sim


def test_variable_batch_size_reaches_256_rows(wide_engine):
    """Token budget 256 x 16 with cells of 16: allowance 256 / 128 / 64 rows for the cells 16 / 32 / 48 and the
    base batch 8 from the threshold 64 on (the constants of Sec. 4.2 scaled to responses of at most 64 tokens)."""
    from paper_2305_13144_b200 import api
    g = _group(1024, seed=5)
    cfg = api.sched_cfg(bin_size=16, base_batch=8, use_vbs=True, vbs_len_threshold=64, vbs_token_budget=256 * 16,
                        min_batch=8, max_batch=256, max_new_tokens=64)
    res, sim = _run_and_compare(wide_engine, g, cfg)
    sizes = [len(b.rows) for b in sim["batches"] if not b.is_recompute]
    assert max(sizes) == 256 and 128 in sizes and 64 in sizes and 8 in sizes
    assert len(sim["failures"]) > 0                        # the cap cut rows and they were regenerated


def test_kv_budget_cuts_batches(wide_engine):
    """Same switches with a key/value budget of 48 rows x 96 tokens: no batch may need more, so the 256- and
    128-row batches of the previous test are cut short by the admission test, not by the allowance."""
    from paper_2305_13144_b200 import api
    g = _group(512, seed=6)
    budget = 48 * 96 * KV_TOK_TINY
    cfg = api.sched_cfg(bin_size=16, base_batch=8, use_vbs=True, vbs_len_threshold=64, vbs_token_budget=256 * 16,
                        min_batch=8, max_batch=256, max_new_tokens=64, kv_budget_bytes=budget,
                        kv_bytes_per_token=KV_TOK_TINY)
    res, sim = _run_and_compare(wide_engine, g, cfg)
    first = [b for b in sim["batches"] if not b.is_recompute]
    cut = [b for b in first if len(b.rows) < osch.vbs_batch(max(osch.bin_of(g.pred_len[r], oracle_sched_cfg(cfg))
                                                                 for r in b.rows), oracle_sched_cfg(cfg))]
    assert len(cut) >= 3                                   # the budget, not the allowance, ended these batches
    for b in first:
        assert len(b.rows) * (max(int(g.prompt_len[r]) for r in b.rows) + b.cap) * KV_TOK_TINY <= budget or len(b.rows) == 1


@pytest.mark.parametrize("switches", [dict(use_fcr=False), dict(bin_size=1), dict(bin_size=1, use_fcr=False),
                                      dict(bin_size=1, use_vbs=True)])
def test_table5_switches(wide_engine, switches):
    """FCR off (caps at max_new, no failures), no binning (cell 1), both, and no binning under VBS."""
    from paper_2305_13144_b200 import api
    g = _group(200, seed=7)
    kw = dict(bin_size=16, base_batch=8, use_vbs=False, use_fcr=True, vbs_len_threshold=64,
              vbs_token_budget=256 * 16, min_batch=8, max_batch=256, max_new_tokens=64)
    kw.update(switches)
    res, sim = _run_and_compare(wide_engine, g, api.sched_cfg(**kw))
    if not kw["use_fcr"]:
        assert sim["failures"] == [] and all(b.cap == 64 for b in sim["batches"])


def test_natural_eos_group_matches_oracle_decoder_and_scheduler():
    """No forced lengths (eos_at = NULL): a row ends when its arg-max is the EOS id, the engine polls the number
    of active rows between chunks of decode steps, and FCR cuts and regenerates rows as usual.

    A free-running row can only be compared with the oracle while no decision is a near-tie, so the group is
    chosen on the ORACLE side: of up to 900 seeded candidate prompts, the first 96 whose every arg-max (the oracle's
    float64 logits) leads the runner-up by more than twice the logit tolerance.  For those the engine must
    reproduce the oracle decoder's tokens, lengths and statuses exactly, and -- with the oracle's lengths as the
    true lengths -- the scheduler oracle's batch log.  To make EOS a likely arg-max and the lengths varied, the
    vocabulary has 64 words, the weights are drawn four times wider than usual (so that the context, not only
    the last token, decides the next one) and the EOS row of the LM head is scaled by 1.5."""
    from paper_2305_13144_b200 import api
    shape = synth.ModelShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=64)
    w = synth.make_weights(shape, seed=99, sigma=0.08)
    w["lm_head"][shape.eos_id] = synth.round_to_bf16(w["lm_head"][shape.eos_id] * 1.5)
    model = oracle_model(shape, w)
    max_new, want = 24, 96
    rng = np.random.default_rng(3)
    prompts, refs = [], []
    for _ in range(900):
        p = rng.integers(3, shape.vocab, size=int(rng.integers(4, 20))).tolist()
        r = od.generate(model, p, max_new, None, keep_logits=True)
        clear = True
        for lg in r["logits"]:
            top = np.sort(lg)[-2:]
            if top[1] - top[0] <= 2 * LOGIT_TOL * np.max(np.abs(lg)):
                clear = False
                break
        if clear:
            prompts.append(p)
            refs.append(r)
            if len(prompts) == want:
                break
    assert len(prompts) == want
    true_len = np.array([len(r["tokens"]) for r in refs], dtype=np.int32)
    assert (true_len < max_new).sum() >= want // 2 and len(set(true_len.tolist())) > 8     # EOS does happen, at varied lengths
    off = np.zeros(want + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(p) for p in prompts])
    toks = np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts])
    noise = np.rint(3.0 * rng.standard_normal(want)).astype(np.int32)
    pred = np.clip(true_len + noise, 1, max_new).astype(np.int32)
    eng = engine(shape, w, max_batch=16, max_ctx=64, max_prefill=512, max_new=max_new, kv_tokens=16 * 64)
    plen = np.array([len(p) for p in prompts], dtype=np.int32)
    for vanilla in (False, True):
        cfg = api.sched_cfg(bin_size=4, base_batch=8, max_new_tokens=max_new, vanilla=vanilla)
        perm = synth.make_permutation(want, 1) if vanilla else None
        res = api.ss_run_group(eng, cfg, toks, off, pred, perm, None)
        assert api.ss_last_device_status(eng) == 0
        for i, r in enumerate(refs):
            assert res["len"][i] == len(r["tokens"]), i
            assert res["tokens"][i, :res["len"][i]].tolist() == r["tokens"], i
            assert bool(res["status"][i]) == r["finished"], i
        sim = osch.simulate(plen, pred, true_len, oracle_sched_cfg(cfg), perm)
        assert_group_matches_simulation(res, sim, want, true_len, shape.eos_id)


def test_perception_pass_at_its_batch_size():
    """The length-perception pass as a workload (Sec. 4.1 "Overhead of Length Prediction"; App. A: the predictor's
    answer is a few tokens after the instruction): every query's prompt plus one fixed instruction suffix goes
    through the prompt pass and three tokens are generated, in batches of 256, through ss_run_group().  The batch
    log must equal the scheduler oracle's, and the two free tokens of 32 sampled rows must equal the oracle
    decoder's wherever its decision is clear (top-2 gap above twice the logit tolerance)."""
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    eng = engine(shape, w, max_batch=256, max_ctx=128, max_prefill=16384, max_new=8, kv_tokens=256 * 64)
    g = _group(600, seed=11)
    rng = np.random.default_rng(11)
    suffix = rng.integers(3, shape.vocab, size=12).astype(np.int32)
    plen = g.prompt_len + len(suffix)
    off = np.zeros(g.n + 1, dtype=np.int64)
    off[1:] = np.cumsum(plen)
    toks = np.concatenate([np.concatenate([g.prompt(i), suffix]) for i in range(g.n)]).astype(np.int32)
    three = np.full(g.n, 3, dtype=np.int32)
    cfg = api.sched_cfg(vanilla=True, base_batch=256, max_new_tokens=4)
    res = api.ss_run_group(eng, cfg, toks, off, three, np.arange(g.n, dtype=np.int32), three)
    sim = osch.simulate(plen, three, three, oracle_sched_cfg(cfg), list(range(g.n)))
    assert_group_matches_simulation(res, sim, g.n, three, shape.eos_id)
    assert [len(b.rows) for b in sim["batches"]] == [256, 256, 88]
    model = oracle_model(shape, w)
    clear = 0
    for i in range(0, g.n, 19):                             # 32 rows, spread over the three batches
        ref = od.generate(model, toks[off[i]:off[i + 1]].tolist(), 4, 3, keep_logits=True)
        assert res["tokens"][i, 2] == shape.eos_id
        for t in range(2):
            lg = ref["logits"][t].copy()
            lg[shape.eos_id] = -np.inf
            top = np.sort(lg)[-2:]
            if top[1] - top[0] > 2 * LOGIT_TOL * np.max(np.abs(ref["logits"][t])):
                assert res["tokens"][i, t] == ref["tokens"][t], (i, t)
                clear += 1
            else:
                break                                       # after a near-tie the histories may differ
    assert clear >= 30                                      # 33 of the 64 decisions are clear on the oracle side


def test_batch_lists_dealt_to_replicas_reproduce_the_single_engine_run(wide_engine):
    """ss_run_batches() + the replica dispatch with two "replicas" played one after the other by the same
    engine: the assembled result (order, failures, log, every token) equals ss_run_group()'s on one GPU."""
    from paper_2305_13144_b200 import api
    from paper_2305_13144_b200.replicas import run_group_replicas
    eng = wide_engine
    g = _group(300, seed=9)
    cfg = api.sched_cfg(bin_size=16, base_batch=8, use_vbs=True, vbs_len_threshold=64, vbs_token_budget=256 * 16,
                        min_batch=8, max_batch=256, max_new_tokens=64)
    whole = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, None, g.true_len)

    def run(order, batches):
        return api.ss_run_batches(eng, cfg, g.prompt_tokens, g.prompt_off, g.true_len, order, batches)

    # two ranks as two threads: the exchange is a barrier, and the one engine serves one of them at a time
    import threading
    world = 2
    lock, barrier = threading.Lock(), threading.Barrier(world)
    box, results, errors = [None] * world, [None] * world, []

    def locked_run(order, batches):
        with lock:
            return run(order, batches)

    def rank_main(rank):
        def gather(obj):
            box[rank] = obj
            barrier.wait(timeout=120)
            got = list(box)
            barrier.wait(timeout=120)
            return got
        try:
            results[rank] = run_group_replicas(api, cfg, g, None, rank=rank, world=world, run_batches=locked_run,
                                               gather=gather, shape=synth.TINY)
        except Exception as e:                              # let the other thread out of its barrier
            errors.append(e)
            barrier.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    for res in results:
        assert res["order"].tolist() == whole["order"].tolist()
        assert (res["tokens"] == whole["tokens"]).all() and (res["len"] == whole["len"]).all()
        assert (res["status"] == whole["status"]).all()
        assert [(b["first_row"], b["n_rows"], b["cap"], b["is_recompute"], b["steps"], b["n_failed"]) for b in res["log"]] == \
               [(b["first_row"], b["n_rows"], b["cap"], b["is_recompute"], b["steps"], b["n_failed"]) for b in whole["log"]]
        assert {b["gpu"] for b in res["log"]} == {0, 1}
        for k in ("useful_tokens", "row_steps", "steps"):
            assert res["stats"][k] == whole["stats"][k]
