"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Tolerances (bf16 storage of weights, activations and cache; fp32 accumulation):
per-step logits, teacher-forced on the oracle's tokens, max-abs error <= 2e-2 * max|logit|;
final hidden state relative L2 <= 1e-2.  Integer results (schedules, lengths, status) bit-exact.
"""
import numpy as np
import pytest

from oracle import decoder as od
from oracle import scheduler as osch
from paper_2305_13144_b200 import synth

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
HIDDEN_TOL = 1e-2


def _oracle(shape, w):
    return od.Decoder(w, n_layers=shape.n_layers, n_heads=shape.n_heads, head_dim=shape.head_dim,
                      rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, eos_id=shape.eos_id)


def _engine(shape, w, *, max_batch=16, max_ctx=128, max_prefill=512, max_new=64, kv_tokens=4096):
    from paper_2305_13144_b200 import api
    rt = api.runtime_cfg(max_batch, max_ctx, max_prefill, max_new, kv_tokens)
    bits = {k: synth.to_bf16_bits(v) for k, v in w.items()}
    return api.make_engine(shape, rt, bits)


def _teacher_forced(shape, w, prompts, targets, cap, eng=None, **kw):
    """Runs oracle and GPU side by side; returns worst relative logit error and hidden rel-L2."""
    import torch
    from paper_2305_13144_b200 import api
    model = _oracle(shape, w)
    B = len(prompts)
    ref = [od.generate(model, p, cap, int(t), keep_logits=True, keep_hidden=True) for p, t in zip(prompts, targets)]
    eng = eng or _engine(shape, w, **kw)
    toks = np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts])
    cu = np.zeros(B + 1, dtype=np.int32)
    cu[1:] = np.cumsum([len(p) for p in prompts])
    dl = torch.zeros(B, shape.vocab, dtype=torch.float32, device="cuda")
    dh = torch.zeros(B, shape.d_model, dtype=torch.float32, device="cuda")
    nxt = torch.zeros(B, dtype=torch.int32, device="cuda")
    steps = max(len(r["tokens"]) for r in ref)
    worst_logit, worst_hidden = 0.0, 0.0
    for t in range(steps):
        alive = [r for r in range(B) if len(ref[r]["tokens"]) > t]
        forced = torch.tensor([ref[r]["tokens"][t] if r in alive else shape.eos_id for r in range(B)],
                              dtype=torch.int32, device="cuda")
        if t == 0:
            api.ss_prefill(eng, toks, cu, targets, cap, forced_tokens=forced, dump_logits=dl, dump_hidden=dh,
                           first_tokens=nxt)
        else:
            api.ss_decode_step(eng, forced_tokens=forced, dump_logits=dl, dump_hidden=dh, next_tokens=nxt)
        torch.cuda.synchronize()
        assert api.ss_last_device_status(eng) == 0
        gl, gh, gn = dl.cpu().numpy(), dh.cpu().numpy(), nxt.cpu().numpy()
        for r in range(B):
            if r in alive:
                rl, rh = ref[r]["logits"][t], ref[r]["hidden"][t]
                worst_logit = max(worst_logit, float(np.max(np.abs(gl[r] - rl)) / np.max(np.abs(rl))))
                worst_hidden = max(worst_hidden, float(np.linalg.norm(gh[r] - rh) / np.linalg.norm(rh)))
                assert gn[r] == ref[r]["tokens"][t]
            else:
                assert gn[r] == shape.eos_id           # finished rows report EOS and cost nothing
    out, lens, status = api.ss_read_batch(eng, B, cap)
    for r in range(B):
        assert lens[r] == len(ref[r]["tokens"])
        assert out[r, :lens[r]].tolist() == ref[r]["tokens"]
        assert bool(status[r]) == ref[r]["finished"]
    api.ss_release_batch(eng)
    return worst_logit, worst_hidden


@pytest.mark.parametrize("n_layers", [0, 1, 2])
def test_tiny_teacher_forced_logits_and_hidden(n_layers):
    shape = synth.TINY.with_layers(n_layers)
    w = synth.make_weights(shape, seed=1234)
    g = synth.group_tiny(seed=0)
    rows = [0, 1, 2, 3, 4, 5, 6, 7]
    prompts = [g.prompt(i).tolist() for i in rows]
    targets = [min(int(g.true_len[i]), 10) for i in rows]
    targets[1], targets[5] = 1, 3                          # a row that ends in the prompt pass, a short one
    el, eh = _teacher_forced(shape, w, prompts, targets, cap=8)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (el, eh)


def test_tiny_ragged_batch_sizes_and_page_boundaries():
    """Batch sizes that are not multiples of the token tile, prompts that end exactly on a page
    boundary (32 tokens) and decoding across it."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    eng = _engine(shape, w, max_batch=32, max_ctx=160)
    rng = np.random.default_rng(5)
    for B in (1, 3, 17):
        lens = [31, 32, 33][:B] + [int(x) for x in rng.integers(8, 40, size=max(0, B - 3))]
        prompts = [(rng.integers(3, shape.vocab, size=n)).tolist() for n in lens]
        targets = [int(x) for x in rng.integers(2, 6, size=B)]
        el, eh = _teacher_forced(shape, w, prompts, targets, cap=5, eng=eng)
        assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (B, el, eh)


def test_very_short_prompts_leave_attention_groups_without_keys():
    """Fewer cached tokens than key groups in the decode-attention CTA (prompts of 1, 2, 5 tokens)."""
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    rng = np.random.default_rng(11)
    prompts = [rng.integers(3, shape.vocab, size=n).tolist() for n in (1, 2, 5, 9, 14, 30)]
    el, eh = _teacher_forced(shape, w, prompts, [6, 6, 5, 4, 6, 3], cap=6)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (el, eh)


def test_long_context_spans_attention_chunks():
    """A prompt longer than one attention work item (256 tokens) and one prompt-pass query tile."""
    shape = synth.TINY.with_layers(1)
    w = synth.make_weights(shape, seed=77)
    rng = np.random.default_rng(9)
    prompts = [rng.integers(3, shape.vocab, size=n).tolist() for n in (300, 257, 40)]
    el, eh = _teacher_forced(shape, w, prompts, [4, 3, 4], cap=4, max_ctx=384, max_prefill=1024)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (el, eh)


def test_graph_replay_equals_single_steps_and_free_running_matches_oracle_mostly():
    import torch
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    g = synth.group_tiny(seed=2)
    rows = list(range(8))
    toks = np.concatenate([g.prompt(i) for i in rows]).astype(np.int32)
    cu = np.zeros(9, dtype=np.int32)
    cu[1:] = np.cumsum([g.prompt_len[i] for i in rows])
    targets = np.array([int(g.true_len[i]) for i in rows], dtype=np.int32)
    cap = 24
    eng = _engine(shape, w)
    pinned = torch.zeros(1, dtype=torch.int32).pin_memory()
    results = []
    for mode in ("steps", "graph"):
        api.ss_prefill(eng, toks, cu, targets, cap)
        if mode == "steps":
            for _ in range(cap - 1):
                api.ss_decode_step(eng, n_active_host=pinned)
        else:
            api.ss_decode_steps(eng, cap - 1, n_active_host=pinned)
        torch.cuda.synchronize()
        results.append(api.ss_read_batch(eng, 8, cap))
        assert int(pinned[0]) == 0
        api.ss_release_batch(eng)
    (t0, l0, s0), (t1, l1, s1) = results
    assert (t0 == t1).all() and (l0 == l1).all() and (s0 == s1).all()        # deterministic, graph == eager
    assert l0.tolist() == np.minimum(targets, cap).tolist()
    assert s0.tolist() == [int(t <= cap) for t in targets]
    # free-running tokens: bf16 may flip a near-tie, after which a row legitimately diverges;
    # the first token of every row and the large majority of all tokens must agree
    model = _oracle(shape, w)
    agree = total = 0
    for r, i in enumerate(rows):
        ref = od.generate(model, g.prompt(i).tolist(), cap, int(targets[r]))["tokens"]
        assert t0[r, 0] == ref[0]
        agree += int((t0[r, :len(ref)] == np.array(ref)).sum())
        total += len(ref)
        n = l0[r]
        assert shape.eos_id not in t0[r, :n - 1].tolist()
        assert (t0[r, n - 1] == shape.eos_id) == bool(s0[r])
    assert agree / total > 0.8


def test_run_group_log_is_bit_exact_with_scheduler_oracle():
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    eng = _engine(shape, w, max_batch=16, max_ctx=128, max_new=64, kv_tokens=8 * 128)
    for seed in (0, 1):
        g = synth.group_tiny(seed)
        for vanilla in (False, True):
            cfg = api.sched_cfg(bin_size=16, base_batch=8, max_new_tokens=64, vanilla=vanilla)
            perm = synth.make_permutation(g.n, seed) if vanilla else None
            res = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, perm, g.true_len)
            ocfg = osch.SchedCfg(bin_size=16, base_batch=8, max_new_tokens=64, vanilla=vanilla)
            sim = osch.simulate(g.prompt_len, g.pred_len, g.true_len, ocfg, perm)
            order = res["order"]
            assert order[:g.n].tolist() == sim["order"]
            nf = len(sim["failures"])
            assert order[g.n:g.n + nf].tolist() == sim["failures"] and (order[g.n + nf:] == -1).all()
            assert len(res["log"]) == len(sim["batches"])
            for rec, ob in zip(res["log"], sim["batches"]):
                rows = order[rec["first_row"]:rec["first_row"] + rec["n_rows"]].tolist()
                assert rows == ob.rows and rec["cap"] == ob.cap and rec["is_recompute"] == int(ob.is_recompute)
                assert rec["steps"] == ob.steps and rec["n_failed"] == len(ob.failed)
            assert res["len"].tolist() == g.true_len.tolist()              # every row finally reaches its EOS
            assert res["status"].tolist() == [1] * g.n
            st = res["stats"]
            assert st["useful_tokens"] == sim["useful_tokens"] and st["row_steps"] == sim["row_steps"]
            assert st["steps"] == sim["steps"] and st["n_failed"] == nf
            for i in range(g.n):
                assert res["tokens"][i, g.true_len[i] - 1] == shape.eos_id
            assert st["kernel_launches"] > 0


def test_errors_before_launch():
    from paper_2305_13144_b200 import api
    shape = synth.TINY.with_layers(1)
    w = synth.make_weights(shape, seed=1)
    eng = _engine(shape, w, max_batch=4, max_ctx=64, max_new=16, kv_tokens=64)
    toks = np.arange(3, 23, dtype=np.int32)
    with pytest.raises(api.SSError) as e:
        api.ss_decode_step(eng)
    assert e.value.code == api.SS_ERR_STATE
    with pytest.raises(api.SSError) as e:            # 5 rows > max_batch
        api.ss_prefill(eng, toks, [0, 4, 8, 12, 16, 20], None, 4)
    assert e.value.code == api.SS_ERR_CAPACITY
    with pytest.raises(api.SSError) as e:            # pool of 64 tokens (+4 slack pages) cannot hold 4 x (40+16)
        api.ss_prefill(eng, np.tile(toks, 8), [0, 40, 80, 120, 160], None, 16)
    assert e.value.code == api.SS_ERR_KV_BUDGET
    with pytest.raises(api.SSError) as e:            # token id out of range
        api.ss_prefill(eng, np.array([5, shape.vocab], dtype=np.int32), [0, 2], None, 4)
    assert e.value.code == api.SS_ERR_ARG
    api.ss_prefill(eng, toks, [0, 20], None, 4)      # still usable afterwards
    api.ss_release_batch(eng)


@pytest.mark.parametrize("B", [40, 64, 100, 130])
def test_wide_batches_span_several_token_tiles(B):
    """Batches wider than 16 rows: token tiles of 48 and 64 (64-lane accumulator, all four lane quarters),
    112 (one 128-lane accumulator tile) and 144 (two 128-lane tiles); the per-tile arg-max in groups of 64
    rows; attention passes of more than 8 (row, head) pairs per CTA."""
    shape = synth.TINY.with_layers(1)
    w = synth.make_weights(shape, seed=21)
    rng = np.random.default_rng(B)
    lens = rng.integers(3, 70, size=B)
    prompts = [rng.integers(3, shape.vocab, size=int(n)).tolist() for n in lens]
    targets = [int(x) for x in rng.integers(1, 4, size=B)]
    el, eh = _teacher_forced(shape, w, prompts, targets, cap=3, max_batch=256, max_ctx=128, max_prefill=8192,
                             max_new=8, kv_tokens=256 * 96)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (B, el, eh)


def test_wide_ffn_reads_tile_tables_from_global_memory():
    """A feed-forward width whose gate/up projection alone has 248 tiles of 256 rows: the four per-layer
    tile tables (258 entries) no longer fit the decode kernel's shared-memory copy, so every stage looks its
    partial segments up in global memory.  Head size 128, one layer, ragged batch of 5."""
    shape = synth.ModelShape(n_layers=1, d_model=512, n_heads=4, head_dim=128, d_ffn=31744, vocab=1024)
    w = synth.make_weights(shape, seed=33)
    rng = np.random.default_rng(33)
    prompts = [rng.integers(3, shape.vocab, size=int(n)).tolist() for n in (9, 33, 17, 40, 5)]
    targets = [4, 2, 4, 3, 1]
    el, eh = _teacher_forced(shape, w, prompts, targets, cap=4, max_batch=16, max_ctx=64, max_prefill=256,
                             max_new=8, kv_tokens=1024)
    assert el <= LOGIT_TOL and eh <= HIDDEN_TOL, (el, eh)


def test_7b_shape_two_layers_sampled_rows():
    """The 7B shape (d 4096, 32 heads x 128, FFN 11008, vocab 32000) cut to two layers, batch 16 with the
    benchmark's prompt lengths; the oracle follows the three rows with the shortest prompts through the
    prompt pass and two decode steps; all rows run free, and a row is compared for as long as its tokens
    agree with the oracle's (a disagreement is only accepted on a near-tie of the oracle's top two logits).

    Hidden-state tolerance here is 2e-2, not the 1e-2 of the small configuration: with N(0, 0.02) weights at
    d = 4096 the projections' outputs (std ~0.4) dwarf the embedding (std 0.02), so the residual stream's
    relative error IS the relative error of the bf16 operand chain.  Re-running the oracle's own arithmetic
    with nothing changed but a round-to-bf16 at the operands the GPU stores in bf16 (normalised input,
    q/k/v, attention output, SwiGLU output) gives 1.1e-2 on this input, 1.35e-2 with the prompt pass's two
    extra roundings (q/k/v and gate/up leave its GEMMs as bf16) -- the floor of the format, not of the kernels."""
    import torch
    from paper_2305_13144_b200 import api
    shape = synth.LLAMA_7B.with_layers(2)
    w = synth.make_weights(shape, seed=7)
    g = synth.group_7b_batch16(seed=0)
    B = g.n
    rows = np.argsort(g.prompt_len)[:3].tolist()
    model = od.Decoder(w, n_layers=2, n_heads=shape.n_heads, head_dim=shape.head_dim, rms_eps=shape.rms_eps,
                       rope_theta=shape.rope_theta, eos_id=shape.eos_id, dtype=np.float64)
    steps = 3
    ref = {r: od.generate(model, g.prompt(r).tolist(), steps, steps + 5, keep_logits=True, keep_hidden=True) for r in rows}
    del model
    eng = api.make_engine(shape, api.runtime_cfg(16, 768, 4096, 512, 16 * 768),
                          {k: synth.to_bf16_bits(v) for k, v in w.items()})
    cu = np.zeros(B + 1, dtype=np.int32)
    cu[1:] = np.cumsum(g.prompt_len)
    dl = torch.zeros(B, shape.vocab, dtype=torch.float32, device="cuda")
    dh = torch.zeros(B, shape.d_model, dtype=torch.float32, device="cuda")
    nxt = torch.zeros(B, dtype=torch.int32, device="cuda")
    worst_l = worst_h = 0.0
    for t in range(steps):
        if t == 0:
            api.ss_prefill(eng, g.prompt_tokens, cu, np.full(B, steps + 5, dtype=np.int32), 512,
                           dump_logits=dl, dump_hidden=dh, first_tokens=nxt)
        else:
            api.ss_decode_step(eng, dump_logits=dl, dump_hidden=dh, next_tokens=nxt)
        torch.cuda.synchronize()
        assert api.ss_last_device_status(eng) == 0
        gl, gh, gn = dl.cpu().numpy(), dh.cpu().numpy(), nxt.cpu().numpy()
        for r in rows:
            rl, rh = ref[r]["logits"][t], ref[r]["hidden"][t]
            worst_l = max(worst_l, float(np.max(np.abs(gl[r] - rl)) / np.max(np.abs(rl))))
            worst_h = max(worst_h, float(np.linalg.norm(gh[r] - rh) / np.linalg.norm(rh)))
            # free running: the argmax must agree unless the oracle's top two logits are within the tolerance
            top2 = np.sort(rl)[-2:]
            if top2[1] - top2[0] > 2 * LOGIT_TOL * np.max(np.abs(rl)):
                assert gn[r] == ref[r]["tokens"][t]
        if any(gn[r] != ref[r]["tokens"][t] for r in rows):
            break                                    # histories diverged on a near-tie: nothing more to compare
    assert t >= 1
    assert worst_l <= LOGIT_TOL and worst_h <= 2e-2, (worst_l, worst_h)
    api.ss_release_batch(eng)


def test_full_size_7b_zero_output_projections_closed_form():
    """All 32 layers at the benchmark's shapes and launch configuration.  With Wo = 0 and Wdown = 0 every
    layer runs (projections, cache, attention) but leaves the residual stream at the embedding, so
    logits = Wlm . RMSNorm(E[token]) -- which the oracle evaluates for sampled (row, vocabulary id)."""
    import torch
    import bench
    from paper_2305_13144_b200 import api
    shape = synth.LLAMA_7B
    rt = api.runtime_cfg(16, 768, 4096, 512, 16 * 768)
    m = api.model_cfg(shape)
    arena = torch.empty(api.ss_arena_bytes(m, rt) + 1024, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    eng = api.ss_create(m, rt, arena, torch.cuda.Stream())
    keep = {}
    for name, t in bench.device_weights(shape, 99, "cuda:0"):
        if name.endswith(".wo") or name.endswith(".w_down"):
            t.zero_()
        if name in ("embed", "lm_head", "final_norm"):
            keep[name] = t
        api.ss_load_weights(eng, {name: t})
    g = synth.group_7b_batch16(seed=1)
    B = g.n
    cu = np.zeros(B + 1, dtype=np.int32)
    cu[1:] = np.cumsum(g.prompt_len)
    rng = np.random.default_rng(5)
    dl = torch.zeros(B, shape.vocab, dtype=torch.float32, device="cuda")
    fed = np.array([g.prompt(r)[-1] for r in range(B)])          # token whose embedding the logits come from
    for t in range(3):
        forced_np = rng.integers(3, shape.vocab, size=B).astype(np.int32)
        forced = torch.from_numpy(forced_np).cuda()
        if t == 0:
            api.ss_prefill(eng, g.prompt_tokens, cu, np.full(B, 100, dtype=np.int32), 512, forced_tokens=forced,
                           dump_logits=dl)
        else:
            api.ss_decode_step(eng, forced_tokens=forced, dump_logits=dl)
        torch.cuda.synchronize()
        assert api.ss_last_device_status(eng) == 0
        got = dl.cpu().numpy()
        E = keep["embed"][torch.from_numpy(fed).cuda().long()].float().cpu().numpy().astype(np.float64)
        vs = rng.integers(0, shape.vocab, size=64)
        Wl = keep["lm_head"][torch.from_numpy(vs).cuda().long()].float().cpu().numpy().astype(np.float64)
        gain = keep["final_norm"].float().cpu().numpy().astype(np.float64)
        for r in range(B):
            exp = od.rmsnorm(E[r], gain, shape.rms_eps) @ Wl.T
            scale = np.max(np.abs(got[r]))
            assert np.max(np.abs(got[r, vs] - exp)) <= LOGIT_TOL * scale, (t, r)
        fed = forced_np
    api.ss_release_batch(eng)
