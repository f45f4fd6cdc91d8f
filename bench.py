#!/usr/bin/env python
"""Benchmark of the sequence-scheduling decode engine.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--no-group]

One "step" = one pass of the whole hot path over one micro-batch: ss_run_group() on the
LLaMA-7B-shaped decoder (random bf16 weights) with a single vanilla micro-batch of 16 queries
(prompts U[64,256], response lengths lognormal(median 120, sigma 0.7) clipped to 512, ended by a
forced EOS): schedule, prompt pass, decode steps until every row has finished, read-back.
`value` is generated (useful) tokens per second from the device-timed phases (CUDA events
around the prompt pass and the decode loop, inputs resident); `e2e` is the same metric over the
wall clock of the C-ABI call with host buffers in and out.  `roofline` is the decode loop's
algorithmic HBM bytes (weights once per step + cached keys/values of the active rows + the
entries written) over its device time, against the measured copy bandwidth.
After the timed steps (N = 1) the 1024-query group is run once per arm -- vanilla random batching,
sequence scheduling with FCR, and FCR + variable batch size -- and reported under "group" with the
gain over vanilla; each arm's batch log is checked against the scheduler oracle (--no-group skips this).

N > 1: the path does not shard (one GPU per engine), so ranks run independent replicas on
different seeds; value = tokens of all ranks / slowest rank's time.  Without a launcher in the
environment, --gpus N starts the N worker processes itself.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2305_13144_b200 import synth  # noqa: E402

METRIC = "generated tokens/s"
WORKLOAD = "llama7b-shape bf16, one vanilla micro-batch of 16, prompts U[64,256], responses lognormal(120,0.7)<=512"
L2_NOTE = "inputs larger than L2 (13.2 GB of weights re-read every decode step)"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
KERNEL_SOURCES = ("ss_decode_mega.cuh", "ss_gemm.cuh", "ss_kernels.cuh", "ss_internal.h")


def kernel_sources_sha16() -> str:
    """Fingerprint of the decode kernel's sources, to tell whether stored profiler counters still describe it."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2305_13144_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic_bytes():
    """DRAM bytes (read + write) of one decode-step launch as counted by the profiler, or None when no
    capture of the kernel as it stands now has been recorded (the record carries the sources' fingerprint)."""
    p = os.path.join(ROOT, "profiles", "decode_step_mega_7b_shape_traffic.json")
    try:
        with open(p) as f:
            rec = json.load(f)
        if rec.get("kernel_sources_sha16") == kernel_sources_sha16():
            return float(rec["dram_bytes_per_launch"])
    except Exception:
        pass
    return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def device_weights(shape, seed, device):
    """Random N(0, 0.02) bf16 weights drawn on the device (torch is only the RNG and the memory)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab

    def rnd(*s):
        return (torch.randn(*s, generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)

    yield "embed", rnd(V, d)
    for l in range(shape.n_layers):
        p = f"l{l}."
        yield p + "attn_norm", torch.ones(d, device=device, dtype=torch.bfloat16)
        for k in ("wq", "wk", "wv", "wo"):
            yield p + k, rnd(d, d)
        yield p + "ffn_norm", torch.ones(d, device=device, dtype=torch.bfloat16)
        yield p + "w_gate", rnd(F, d)
        yield p + "w_up", rnd(F, d)
        yield p + "w_down", rnd(d, F)
    yield "final_norm", torch.ones(d, device=device, dtype=torch.bfloat16)
    yield "lm_head", rnd(V, d)


def make_engine(shape, rt, seed, device):
    import torch
    from paper_2305_13144_b200 import api
    m = api.model_cfg(shape)
    nbytes = api.ss_arena_bytes(m, rt)
    arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    torch.cuda.synchronize()
    eng = api.ss_create(m, rt, arena, torch.cuda.Stream())
    for name, t in device_weights(shape, seed, device):
        api.ss_load_weights(eng, {name: t})
    return eng


def _oracle_sample():
    """The oracle as it stands (numpy, fp32 here) on a bounded sample of the benchmark workload: all 16 rows of
    the batch, 16 generated tokens each (prompt pass included), on the 7B shape cut to 1 layer and to 2 layers.
    Returns a closure that runs both once and gives (tokens, seconds scaled to the full depth): the difference
    of the two runs is one layer's time, the rest (embedding, final norm, LM head, token choice) counts once."""
    from oracle import decoder as od
    cap = 16
    g = synth.group_7b_batch16(seed=0)
    prompts = [g.prompt(i).tolist() for i in range(g.n)]
    w2 = synth.make_weights(synth.LLAMA_7B.with_layers(2), seed=1234)
    models = []
    for L_s in (1, 2):
        shape = synth.LLAMA_7B.with_layers(L_s)
        models.append(od.Decoder(w2, n_layers=L_s, n_heads=shape.n_heads, head_dim=shape.head_dim,
                                 rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, eos_id=shape.eos_id,
                                 dtype=np.float32))
    del w2
    L = synth.LLAMA_7B.n_layers

    def run():
        secs, tokens = [], 0
        for m in models:
            t = time.time()
            res = od.run_micro_batch(m, prompts, cap, [cap] * g.n)
            secs.append(time.time() - t)
            tokens = sum(len(r["tokens"]) for r in res["rows"])
        per_layer = max(secs[1] - secs[0], 0.0)
        const = max(secs[0] - per_layer, 0.0)
        return tokens, const + L * per_layer, sum(secs)

    what = (f"all {g.n} rows, {cap} generated tokens each (prompt pass included), timed in fp32 on the 7B shape cut "
            f"to 1 and to 2 layers: one layer's time = the difference, x{L} layers, plus the rest once")
    return run, what


def run_reference(args, rank):
    """The oracle as it stands on the host cores, on a bounded sample of the same workload."""
    if rank != 0:
        return
    t0 = time.time()
    run, what = _oracle_sample()
    setup_s = time.time() - t0
    cores = os.cpu_count()
    times, tokens = [], 0
    for it in range(args.warmup + args.steps):
        tokens, full_s, _ = run()
        if it >= args.warmup:
            times.append(full_s)
    sec = statistics.mean(times)
    value = tokens / sec
    sample = f"{what}; numpy on {cores} threads; setup {setup_s:.0f}s untimed"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": L2_NOTE, "replicas": 1, "layers": synth.LLAMA_7B.n_layers},
            "impl_detail": "cpu oracle (numpy)",
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def cpu_baseline_leg():
    run, what = _oracle_sample()
    tokens, full_s, spent = run()
    cores = os.cpu_count()
    return {"value": tokens / full_s, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"{what}; {spent:.1f}s of CPU time; numpy on {cores} threads"}


def run_cpu_extras():
    """The oracle timed on the host cores beyond the default line's sample: configuration 1 end to end (the small
    model, 32 queries: vanilla batching and sequence scheduling, every micro-batch and the recomputation batches
    generated by the oracle decoder), and the scheduler oracle alone on the groups of configurations 3, 4 and 5."""
    from oracle import decoder as od
    from oracle import scheduler as osch
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    model = od.Decoder(w, n_layers=shape.n_layers, n_heads=shape.n_heads, head_dim=shape.head_dim,
                       rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, eos_id=shape.eos_id)
    g = synth.group_tiny(seed=0)
    out = {"cores": os.cpu_count(), "config1": {}, "scheduler_alone": {}}
    for name, cfg, perm in (("vanilla", osch.SchedCfg(bin_size=16, base_batch=8, max_new_tokens=64, vanilla=True),
                             synth.make_permutation(g.n, 0)),
                            ("scheduled_fcr", osch.SchedCfg(bin_size=16, base_batch=8, max_new_tokens=64), None)):
        sim = osch.simulate(g.prompt_len, g.pred_len, g.true_len, cfg, perm)
        t0 = time.time()
        for b in sim["batches"]:
            res = od.run_micro_batch(model, [g.prompt(r).tolist() for r in b.rows], b.cap, [int(g.true_len[r]) for r in b.rows])
            assert res["steps"] == b.steps
        dt = time.time() - t0
        out["config1"][name] = {"seconds": round(dt, 2), "tokens_per_s": round(sim["useful_tokens"] / dt, 1),
                                "samples_per_s": round(g.n / dt, 2), "steps": sim["steps"], "batches": len(sim["batches"])}
    out["config1"]["gain_vs_vanilla"] = round(out["config1"]["scheduled_fcr"]["tokens_per_s"] /
                                              out["config1"]["vanilla"]["tokens_per_s"], 3)
    kv7 = 2 * synth.LLAMA_7B.d_model * 2 * synth.LLAMA_7B.n_layers
    kv13 = 2 * synth.LLAMA_13B.d_model * 2 * synth.LLAMA_13B.n_layers
    cases = (("config3 (1024 queries, FCR, batch 16)", synth.group_7b_1024(0), osch.SchedCfg()),
             ("config4 (1024 queries, FCR + VBS, 120 GB)", synth.group_7b_1024(0),
              osch.SchedCfg(use_vbs=True, kv_budget_bytes=int(120e9), kv_bytes_per_token=kv7)),
             ("config5 (512 queries, 13B shape, FCR + VBS)", synth.group_13b_512(0),
              osch.SchedCfg(use_vbs=True, max_new_tokens=2048, kv_budget_bytes=int(120e9), kv_bytes_per_token=kv13)))
    for name, grp, cfg in cases:
        reps = 20
        t0 = time.time()
        for _ in range(reps):
            sim = osch.simulate(grp.prompt_len, grp.pred_len, grp.true_len, cfg)
        out["scheduler_alone"][name] = {"ms": round((time.time() - t0) / reps * 1e3, 2), "batches": len(sim["batches"]),
                                        "steps": sim["steps"]}
    return out


def aggregate(tokens_local: float, seconds_local: float, dist):
    """Whole-job numbers from per-rank ones: tokens add up, time is the slowest rank's."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return tokens_local, seconds_local
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([tokens_local], dtype=torch.float64, device=dev)
    s = torch.tensor([seconds_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(s, op=dist.ReduceOp.MAX)
    return float(t.item()), float(s.item())


def stage_trace(eng, api, g, steps=60):
    """Where one decode step spends its time: the batch's prompt pass, `steps` decode steps, then the stage
    stamps of the last step (ss_step_trace), averaged per projection type (microseconds)."""
    import torch
    cu = np.zeros(g.n + 1, dtype=np.int32)
    cu[1:] = np.cumsum(g.prompt_len)
    api.ss_set_trace(eng, True)
    api.ss_prefill(eng, g.prompt_tokens, cu, g.true_len, 512)
    api.ss_decode_steps(eng, steps)
    torch.cuda.synchronize()
    tr = api.ss_step_trace(eng).astype(np.int64)
    api.ss_release_batch(eng)
    api.ss_set_trace(eng, False)
    tr = tr - tr[0]
    ev = tr[2:].reshape(-1, 4)
    names = ["qkv", "o", "gate_up", "down"]
    acc, cnt, prev = {}, {}, tr[1]
    for i, row in enumerate(ev):
        nm = "lm_head" if i == len(ev) - 1 else names[i % 4]
        d = np.array([row[0] - prev, row[1] - row[0], row[2] - row[1], row[3] - row[2]], dtype=np.float64)
        prev = row[3]
        acc[nm] = acc.get(nm, 0) + d
        cnt[nm] = cnt.get(nm, 0) + 1
    out = {"step_us": float(tr[-1]) / 1e3, "after_steps": steps,
           "columns": ["projection_and_drain", "barrier", "following_stage", "barrier"]}
    for nm in acc:
        out[nm] = [round(float(x) / cnt[nm] / 1e3, 2) for x in acc[nm]]
    return out


def check_against_scheduler_oracle(res, g, cfg, perm):
    """Checker (outside every timed region): the batch log the engine reports must equal the scheduler oracle's
    simulation of the same group -- order, failure list, and rows / cap / steps / failures of every batch."""
    from oracle import scheduler as osch
    ocfg = osch.SchedCfg(bin_size=cfg.bin_size, base_batch=cfg.base_batch, use_vbs=bool(cfg.use_vbs),
                         use_fcr=bool(cfg.use_fcr), vbs_len_threshold=cfg.vbs_len_threshold,
                         vbs_token_budget=cfg.vbs_token_budget, min_batch=cfg.min_batch, max_batch=cfg.max_batch,
                         max_new_tokens=cfg.max_new_tokens, kv_budget_bytes=cfg.kv_budget_bytes,
                         kv_bytes_per_token=cfg.kv_bytes_per_token, vanilla=bool(cfg.vanilla))
    sim = osch.simulate(g.prompt_len, g.pred_len, g.true_len, ocfg, perm)
    order, n, nf = res["order"], g.n, len(sim["failures"])
    assert order[:n].tolist() == sim["order"] and order[n:n + nf].tolist() == sim["failures"]
    assert len(res["log"]) == len(sim["batches"])
    for rec, ob in zip(res["log"], sim["batches"]):
        assert order[rec["first_row"]:rec["first_row"] + rec["n_rows"]].tolist() == ob.rows
        assert (rec["cap"], rec["steps"], rec["n_failed"], rec["is_recompute"]) == \
               (ob.cap, ob.steps, len(ob.failed), int(ob.is_recompute))
    assert res["len"].tolist() == g.true_len.tolist()
    return sim


def run_group_arm(eng, api, g, cfg, perm, check=True):
    t0 = time.time()
    res = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, perm, g.true_len)
    wall = time.time() - t0
    if check:
        check_against_scheduler_oracle(res, g, cfg, perm)
    st = res["stats"]
    dev_s = (st["prefill_ms"] + st["decode_ms"]) / 1e3
    return {"tokens_per_s": st["useful_tokens"] / dev_s, "samples_per_s": g.n / dev_s,
            "e2e_tokens_per_s": st["useful_tokens"] / wall, "device_s": dev_s, "wall_s": wall,
            "prefill_s": st["prefill_ms"] / 1e3, "decode_s": st["decode_ms"] / 1e3,
            "batches": st["n_batches"], "steps": st["steps"], "avg_len": st["steps"] / max(1, st["n_batches"]),
            "redundancy": 1.0 - st["useful_tokens"] / max(1, st["row_steps"]),
            "failure_ratio": st["n_failed"] / g.n, "log_equals_scheduler_oracle": bool(check),
            "decode_gbs": st["model_bytes"] / (st["decode_ms"] / 1e3) / 1e9 if st["decode_ms"] > 0 else None}


def run_group_arms_7b(eng, api, kv_tok):
    """Configurations 3 and 4: the 1024-query group at the 7B shape, once per arm -- vanilla random batching,
    sequence scheduling with bins of 50 + FCR at batch 16, and the same with variable batch size (16..256 rows
    inside a 120 GB key/value budget)."""
    g3 = synth.group_7b_1024(seed=0)
    arms = {}
    arms["vanilla"] = run_group_arm(eng, api, g3, api.sched_cfg(vanilla=True), synth.make_permutation(g3.n, 0))
    arms["scheduled_fcr"] = run_group_arm(eng, api, g3, api.sched_cfg(), None)
    arms["scheduled_fcr_vbs"] = run_group_arm(
        eng, api, g3, api.sched_cfg(use_vbs=True, kv_budget_bytes=int(120e9), kv_bytes_per_token=kv_tok), None)
    for k in ("scheduled_fcr", "scheduled_fcr_vbs"):
        arms[k]["gain_vs_vanilla"] = arms[k]["tokens_per_s"] / arms["vanilla"]["tokens_per_s"]
    return {"workload": "llama7b-shape bf16, 1024 queries, prompts U[64,256], responses lognormal(120,0.7)<=512, "
                        "predicted = true + N(0,40), bins of 50", "arms": arms,
            "paper_context": "+86% samples/s on one A100-80G (Table 4), not comparable hardware"}


def run_group_sweep(api, device):
    """Throughput against group size (the paper's Fig. 3b: scheduling needs a group much larger than a micro-batch
    and stops paying at 32): the 1024 queries at the 7B shape are processed in consecutive groups of G, each group
    scheduled on its own (bins of 50 + FCR + variable batch size), against vanilla batching of the same groups."""
    shape = synth.LLAMA_7B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    eng = make_engine(shape, api.runtime_cfg(256, 768, 16384, 512, int(120e9 // kv_tok)), seed=1234, device=device)
    g = synth.group_7b_1024(seed=0)
    perm = synth.make_permutation(g.n, 0)
    points = []
    for G in (32, 64, 128, 256, 512, 1024):
        tot = {"vanilla": [0.0, 0], "scheduled": [0.0, 0]}
        fails = 0
        for lo in range(0, g.n, G):
            ids = np.arange(lo, lo + G)
            off = np.zeros(G + 1, dtype=np.int64)
            off[1:] = np.cumsum(g.prompt_len[ids])
            sub = synth.Group(np.concatenate([g.prompt(i) for i in ids]), off, g.prompt_len[ids], g.true_len[ids],
                              g.pred_len[ids], g.max_new)
            for name, cfg, pm in (("vanilla", api.sched_cfg(vanilla=True), np.argsort(perm[ids]).astype(np.int32)),
                                  ("scheduled", api.sched_cfg(use_vbs=True, kv_budget_bytes=int(120e9),
                                                              kv_bytes_per_token=kv_tok), None)):
                r = run_group_arm(eng, api, sub, cfg, pm)
                tot[name][0] += r["device_s"]
                tot[name][1] += int(sub.true_len.sum())
                if name == "scheduled":
                    fails += int(round(r["failure_ratio"] * G))
        v, sc = tot["vanilla"][1] / tot["vanilla"][0], tot["scheduled"][1] / tot["scheduled"][0]
        points.append({"group_size": G, "vanilla_tokens_per_s": round(v, 1), "scheduled_tokens_per_s": round(sc, 1),
                       "gain_vs_vanilla": round(sc / v, 3), "failure_ratio": round(fails / g.n, 3)})
    return {"metric": METRIC, "unit": "tokens/s", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama7b-shape bf16, 1024 queries in consecutive groups of G; FCR + VBS vs vanilla"},
            "value": points[-1]["scheduled_tokens_per_s"], "points": points,
            "paper_context": "Fig. 3b: throughput grows with the group size and scheduling fails at 32 (one A100-80G)"}


def run_group_dispatch(api, device, rank, world, dist):
    """Configuration 4's group dealt to `world` replicas (paper Sec. 1: micro-batches of different perceived
    lengths go to different GPUs): one schedule, batches dealt longest estimated cost first, failures requeued
    from a shared list; whole-job tokens/s = useful tokens / slowest replica's device time."""
    from paper_2305_13144_b200.replicas import run_group_replicas
    shape = synth.LLAMA_7B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    eng = make_engine(shape, api.runtime_cfg(256, 768, 16384, 512, int(120e9 // kv_tok)), seed=1234, device=device)
    g = synth.group_7b_1024(seed=0)
    cfg = api.sched_cfg(use_vbs=True, kv_budget_bytes=int(120e9), kv_bytes_per_token=kv_tok)

    def gather(obj):
        if world == 1:
            return [obj]
        box = [None] * world
        dist.all_gather_object(box, obj)
        return box

    def run(order, batches):
        return api.ss_run_batches(eng, cfg, g.prompt_tokens, g.prompt_off, g.true_len, order, batches)

    res = run_group_replicas(api, cfg, g, None, rank=rank, world=world, run_batches=run, gather=gather, shape=shape)
    assert res["len"].tolist() == g.true_len.tolist()
    slowest = max(res["device_s"])
    return {"metric": METRIC, "unit": "tokens/s", "n_gpus": world, "dtype": "bf16", "data": "synthetic",
            "scaling": "strong", "higher_is_better": True,
            "config": {"workload": "llama7b-shape bf16, 1024 queries, FCR + VBS, micro-batches dealt to replicas"},
            "value": res["stats"]["useful_tokens"] / slowest, "device_s_per_replica": res["device_s"],
            "batches": res["stats"]["n_batches"], "failure_ratio": res["stats"]["n_failed"] / g.n}


def spawn_replicas(n: int) -> int:
    """`--gpus N` without a launcher: start one worker process per GPU (this script again, with the rank in the
    environment), pass rank 0's JSON line through, return the first non-zero exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def run_group_13b(api, device):
    """Configuration 5: LLaMA-13B shape, 512 queries, prompts U[64,512], responses lognormal(200, 0.7) <= 2048,
    predicted = true + N(0,40), bins of 50; vanilla batching vs FCR + variable batch size in a 120 GB KV budget."""
    shape = synth.LLAMA_13B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    rt = api.runtime_cfg(256, 512 + 2048, 16384, 2048, int(120e9 // kv_tok))
    eng = make_engine(shape, rt, seed=4321, device=device)
    g = synth.group_13b_512(seed=0)
    arms = {}
    arms["vanilla"] = run_group_arm(eng, api, g, api.sched_cfg(vanilla=True, max_new_tokens=2048),
                                    synth.make_permutation(g.n, 0))
    arms["scheduled_fcr_vbs"] = run_group_arm(
        eng, api, g, api.sched_cfg(use_vbs=True, max_new_tokens=2048, kv_budget_bytes=int(120e9),
                                   kv_bytes_per_token=kv_tok), None)
    arms["scheduled_fcr_vbs"]["gain_vs_vanilla"] = arms["scheduled_fcr_vbs"]["tokens_per_s"] / arms["vanilla"]["tokens_per_s"]
    return {"metric": METRIC, "unit": "tokens/s", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama13b-shape bf16, 512 queries, prompts U[64,512], responses lognormal(200,0.7)<=2048"},
            "value": arms["scheduled_fcr_vbs"]["tokens_per_s"], "arms": arms}


def run_ablation(api, device):
    """The three switches of the paper's ablation (Table 5) on the 1024-query group at the 7B shape: sorting by
    predicted length is always on; binning (cells of 50), failure collection and recomputation (FCR), variable
    batch size (VBS).  Vanilla random batching is the reference for the gains."""
    shape = synth.LLAMA_7B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    eng = make_engine(shape, api.runtime_cfg(256, 768, 16384, 512, int(120e9 // kv_tok)), seed=1234, device=device)
    g = synth.group_7b_1024(seed=0)
    arms = {"vanilla": run_group_arm(eng, api, g, api.sched_cfg(vanilla=True), synth.make_permutation(g.n, 0))}
    for binning, fcr, vbs in ((0, 0, 0), (0, 1, 0), (0, 1, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1)):
        cfg = api.sched_cfg(bin_size=50 if binning else 1, use_fcr=bool(fcr), use_vbs=bool(vbs),
                            kv_budget_bytes=int(120e9) if vbs else 0, kv_bytes_per_token=kv_tok if vbs else 0)
        name = "binning=%d fcr=%d vbs=%d" % (binning, fcr, vbs)
        arms[name] = run_group_arm(eng, api, g, cfg, None)
        arms[name]["gain_vs_vanilla"] = arms[name]["tokens_per_s"] / arms["vanilla"]["tokens_per_s"]
    return {"metric": METRIC, "unit": "tokens/s", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama7b-shape bf16, 1024 queries, predicted = true + N(0,40); Table 5 switches"},
            "value": arms["binning=1 fcr=1 vbs=1"]["tokens_per_s"], "arms": arms,
            "paper_context": "Table 5 on one A100-80G: +42 / +44 / +82 / +30 / +52 / +86 % samples/s in the same row order"}


def run_perception(api, device):
    """What the length-perception pass costs against what scheduling gains (the paper's paragraph on the
    overhead of length prediction, Sec. 4.2): every query's prompt plus a 32-token instruction suffix is
    processed and 3 tokens are generated (the predicted number), in batches of 256, before the group is
    scheduled; the predictions themselves are the synthetic ones (true + N(0,40)).  Two variants of the
    generation that follows: prompts recomputed (the paper's choice, App. C), and prompts kept from the
    perception pass as key/value pages from which every generation batch resumes."""
    shape = synth.LLAMA_7B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    budget = int(55e9)                                   # batches; the kept prompts (about 90 GB) share the 150 GB pool
    eng = make_engine(shape, api.runtime_cfg(256, 768, 16384, 512, int(150e9 // kv_tok)), seed=1234, device=device)
    g = synth.group_7b_1024(seed=0)
    sched_cfg = api.sched_cfg(use_vbs=True, kv_budget_bytes=budget, kv_bytes_per_token=kv_tok)
    vanilla = run_group_arm(eng, api, g, api.sched_cfg(vanilla=True), synth.make_permutation(g.n, 0))
    sched = run_group_arm(eng, api, g, sched_cfg, None)
    rng = np.random.Generator(np.random.Philox(7))
    suffix = 32
    plen = g.prompt_len + suffix
    off = np.zeros(g.n + 1, dtype=np.int64)
    np.cumsum(plen, out=off[1:])
    toks = np.empty(int(off[-1]), dtype=np.int32)
    extra = rng.integers(3, shape.vocab, size=suffix).astype(np.int32)         # the same instruction for every query
    for i in range(g.n):
        toks[off[i]:off[i] + g.prompt_len[i]] = g.prompt(i)
        toks[off[i] + g.prompt_len[i]:off[i + 1]] = extra
    three = np.full(g.n, 3, dtype=np.int32)
    cfg = api.sched_cfg(vanilla=True, base_batch=256, max_new_tokens=4)

    def perception_pass():
        t0 = time.time()
        res = api.ss_run_group(eng, cfg, toks, off, three, np.arange(g.n, dtype=np.int32), three)
        st = res["stats"]
        return {"device_s": (st["prefill_ms"] + st["decode_ms"]) / 1e3, "wall_s": time.time() - t0,
                "prefill_s": st["prefill_ms"] / 1e3, "decode_s": st["decode_ms"] / 1e3, "batches": st["n_batches"],
                "steps": st["steps"], "prompt_tokens": int(off[-1])}

    perc = perception_pass()
    # the same pass keeping every query's prompt pages, then the generation resumed from them
    api.ss_set_prompt_cache(eng, 1, g.prompt_len)
    perc_keep = perception_pass()
    api.ss_set_prompt_cache(eng, 2)
    reuse = run_group_arm(eng, api, g, sched_cfg, None)
    api.ss_set_prompt_cache(eng, 0)
    api.ss_drop_prompts(eng)
    useful = float(g.true_len.sum())
    return {"metric": METRIC, "unit": "tokens/s", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama7b-shape bf16, 1024 queries; perception pass = prompt + 32 tokens, 3 generated, batches of 256"},
            "value": useful / (perc["device_s"] + sched["device_s"]),
            "vanilla_tokens_per_s": vanilla["tokens_per_s"], "scheduled_tokens_per_s": sched["tokens_per_s"],
            "perception": perc, "perception_keeping_prompts": perc_keep,
            "scheduled_device_s": sched["device_s"], "vanilla_device_s": vanilla["device_s"],
            "scheduled_from_kept_prompts": {"device_s": reuse["device_s"], "prefill_s": reuse["prefill_s"],
                                            "decode_s": reuse["decode_s"], "steps": reuse["steps"],
                                            "kept_prompt_gb": float(np.ceil(g.prompt_len / 32).sum() * 32 * kv_tok / 1e9)},
            "overhead_of_scheduled_run": perc["device_s"] / sched["device_s"],
            "gain_vs_vanilla_without_perception": sched["tokens_per_s"] / vanilla["tokens_per_s"],
            "gain_vs_vanilla_with_perception": vanilla["device_s"] / (perc["device_s"] + sched["device_s"]),
            "gain_vs_vanilla_with_perception_and_kept_prompts": vanilla["device_s"] / (perc_keep["device_s"] + reuse["device_s"])}


def run_sweep(api, device, peak):
    """Decode-step microbenchmark at the 7B shape over batch size and context (the paper's Fig. 3a / Fig. 6
    axes): every row has the same prompt length, 32 decode steps are timed on the device after 8 warm-up steps;
    bytes = weights + the cached keys/values read + the entries written."""
    import torch
    shape = synth.LLAMA_7B
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    rt = api.runtime_cfg(256, 1024, 16384, 64, 256 * 640)
    eng = make_engine(shape, rt, seed=1234, device=device)
    rng = np.random.default_rng(0)
    out = []
    for ctx in (128, 512):
        for B in (1, 8, 16, 32, 64, 128, 256):
            toks = rng.integers(3, shape.vocab, size=B * ctx, dtype=np.int32)
            cu = (np.arange(B + 1) * ctx).astype(np.int32)
            api.ss_prefill(eng, toks, cu, np.full(B, 1 << 20, dtype=np.int32), 64)
            api.ss_decode_steps(eng, 8)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            st = eng.stream                              # the stream the engine launches on
            n = 32
            e0.record(st)
            api.ss_decode_steps(eng, n)
            e1.record(st)
            e1.synchronize()
            ms = e0.elapsed_time(e1) / n
            api.ss_release_batch(eng)
            ctx_mid = ctx + 8 + n / 2.0                      # cached tokens per row, mid-window
            nbytes = 13214687232 + B * ctx_mid * kv_tok + B * kv_tok
            out.append({"B": B, "ctx": ctx, "ms_per_step": round(ms, 4), "tokens_per_s": round(B / ms * 1e3, 1),
                        "gbs": round(nbytes / ms / 1e6, 1), "frac_of_peak": round(nbytes / ms / 1e6 / peak, 3)})
    return {"metric": "decode step sweep", "unit": "ms/step", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama7b-shape bf16 decode steps, equal-length rows, batch x context sweep"},
            "peak_gbs": peak, "points": out}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-group", action="store_true",
                    help="skip the 1024-query group arms (vanilla vs scheduled) that follow the timed batch-16 steps")
    ap.add_argument("--group-arms", action="store_true", help="kept for old command lines: the arms now run by default")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--trace", action="store_true", help="add the per-stage timing of one decode step")
    ap.add_argument("--group-13b", action="store_true",
                    help="instead of the batch-16 workload: the 13B-shape group of 512 queries, vanilla vs scheduled")
    ap.add_argument("--ablation", action="store_true",
                    help="instead of the batch-16 workload: binning / FCR / VBS switched one by one (1024 queries, 7B shape)")
    ap.add_argument("--perception", action="store_true",
                    help="instead of the batch-16 workload: cost of the length-perception pass against the scheduling gain")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the batch-16 workload: decode-step time over batch size and context (7B shape)")
    ap.add_argument("--group-sweep", action="store_true",
                    help="instead of the batch-16 workload: scheduled vs vanilla over the group size (7B shape)")
    ap.add_argument("--group-dispatch", action="store_true",
                    help="instead of the batch-16 workload: one 1024-query group dealt to the --gpus replicas")
    ap.add_argument("--cpu-extras", action="store_true",
                    help="CPU only: the oracle on configuration 1 end to end and the scheduler oracle on configurations 3-5")
    ap.add_argument("--layers", type=int, default=0, help="debug: truncate the model (invalidates the number)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.cpu_extras:
        if rank == 0:
            print(json.dumps(run_cpu_extras()), flush=True)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))

    import torch
    import torch.distributed as dist
    from paper_2305_13144_b200 import api

    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(device))

    if args.group_dispatch:
        out = run_group_dispatch(api, device, rank, world, dist)
        if rank == 0:
            print(json.dumps(out), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.group_sweep:
        if rank == 0:
            print(json.dumps(run_group_sweep(api, device)), flush=True)
        return
    if args.group_13b:
        if rank == 0:
            print(json.dumps(run_group_13b(api, device)), flush=True)
        return
    if args.ablation:
        if rank == 0:
            print(json.dumps(run_ablation(api, device)), flush=True)
        return
    if args.perception:
        if rank == 0:
            print(json.dumps(run_perception(api, device)), flush=True)
        return
    if args.sweep:
        if rank == 0:
            print(json.dumps(run_sweep(api, device, float(measured_peaks()[0]["hbm_gbs"]))), flush=True)
        return
    shape = synth.LLAMA_7B if not args.layers else synth.LLAMA_7B.with_layers(args.layers)
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    with_group = not args.no_group and not args.layers and world == 1
    if with_group:
        kv_pool = int(120e9 // kv_tok)
        rt = api.runtime_cfg(256, 768, 16384, 512, kv_pool)
    else:
        rt = api.runtime_cfg(16, 768, 4096, 512, 16 * 768)
    eng = make_engine(shape, rt, seed=1234 + rank, device=device)
    g = synth.group_7b_batch16(seed=rank)
    cfg = api.sched_cfg(vanilla=True, base_batch=16, max_new_tokens=512)
    tokens = int(g.true_len.sum())

    def one_step():
        t0 = time.time()
        res = api.ss_run_group(eng, cfg, g.prompt_tokens, g.prompt_off, g.pred_len, None, g.true_len)
        return res, time.time() - t0

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    dev_s = wall_s = decode_s = prefill_s = 0.0
    model_bytes = 0.0
    launches = 0
    steps_dec = 0
    with ClockSampler(local_rank) as clk:
        for _ in range(args.steps):
            res, wall = one_step()
            st = res["stats"]
            dev_s += (st["prefill_ms"] + st["decode_ms"]) / 1e3
            decode_s += st["decode_ms"] / 1e3
            prefill_s += st["prefill_ms"] / 1e3
            wall_s += wall
            model_bytes += st["model_bytes"]
            launches += st["kernel_launches"]
            steps_dec += st["steps"] - st["n_batches"]
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    assert res["len"].tolist() == g.true_len.tolist()
    tok_all, dev_all = aggregate(tokens * args.steps, dev_s, dist if world > 1 else None)
    _, wall_all = aggregate(tokens * args.steps, wall_s, dist if world > 1 else None)

    if rank == 0:
        peaks, which = measured_peaks()
        peak = float(peaks["hbm_gbs"])
        achieved = model_bytes / decode_s / 1e9
        h2d = int(g.prompt_tokens.nbytes + 4 * (g.n + 1) + 4 * g.n + 8 * 4 * 256 + 4 * 16 * 24 + 3 * g.prompt_tokens.nbytes)
        d2h = int(tokens * 4 + 2 * 4 * g.n + 4)
        traffic = measured_traffic_bytes() if shape.n_layers == 32 else None
        line = {
            "metric": METRIC, "value": tok_all / dev_all, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dev_all / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": L2_NOTE, "replicas": world, "layers": shape.n_layers},
            "e2e": {"value": tok_all / wall_all, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "decode_step_mega_kernel (one persistent cooperative launch per decode step)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": which, "peak_nominal": NOMINAL_HBM_GBS, "frac_nominal": achieved / NOMINAL_HBM_GBS,
                         "target_frac": 0.70, "meets_target": bool(achieved / peak >= 0.70), "traffic": traffic,
                         "ms_per_decode_step": decode_s / max(1, steps_dec) * 1e3,
                         "bytes_per_decode_step": model_bytes / max(1, steps_dec)},
            "phases": {"prefill_s_per_step": prefill_s / args.steps, "decode_s_per_step": decode_s / args.steps,
                       "decode_steps_per_step": steps_dec / args.steps},
            "clocks": clk.summary(),
        }
        if args.trace:
            line["stage_trace"] = stage_trace(eng, api, g)
        if with_group:
            line["group"] = run_group_arms_7b(eng, api, kv_tok)
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline_leg()
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
