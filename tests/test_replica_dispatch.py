"""Replica dispatch of one group over several GPUs (Sec. 1 of the paper proposes handing micro-batches of
different perceived lengths to different GPUs): the dealing rule against its oracle and a hand-worked case, and
the whole exchange with two gloo ranks on CPU whose "engine" is the scheduler oracle's arithmetic (a batch runs
min(cap, longest true length) steps; rows longer than a cap below max_new fail).  No GPU."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

from oracle import scheduler as osch
from paper_2305_13144_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KV_TOK = 2 * synth.LLAMA_7B.d_model * 2 * synth.LLAMA_7B.n_layers


def test_deal_hand_worked():
    """Three replicas, weight term 100, 1 byte per cached token, prompts of 10: costs are cap * (100 + rows * (10 +
    cap / 2)): (4 rows, cap 20) -> 20 * 180 = 3600; (2, 40) -> 40 * 160 = 6400; (4, 10) -> 10 * 160 = 1600;
    (1, 60) -> 60 * 140 = 8400; (2, 20) -> 20 * 140 = 2800.  By decreasing cost: 8400 -> replica 0, 6400 -> 1,
    3600 -> 2, 2800 -> 2 (total 6400; a tie with replica 1 would go to the lower one, but 2 is the smallest at
    3600), 1600 -> replica 1 or 2?  loads are 8400, 6400, 6400: the lower replica, 1."""
    batches = [osch.Batch([0, 1, 2, 3], 20), osch.Batch([4, 5], 40), osch.Batch([6, 7, 8, 9], 10),
               osch.Batch([10], 60), osch.Batch([11, 12], 20)]
    assert osch.deal(batches, [10] * 13, 100, 1, 3) == [2, 1, 1, 0, 2]
    assert osch.deal(batches, [10] * 13, 100, 1, 1) == [0] * 5


def test_library_deal_equals_oracle_on_the_evaluation_groups():
    from paper_2305_13144_b200 import api
    from paper_2305_13144_b200.replicas import weight_bytes_per_step
    W = weight_bytes_per_step(synth.LLAMA_7B)
    assert W == 13214687232                                # the 7B shape's weight bytes per decode step
    g = synth.group_7b_1024(seed=1)
    for vbs in (False, True):
        cfg = api.sched_cfg(use_vbs=vbs, kv_budget_bytes=int(120e9) if vbs else 0, kv_bytes_per_token=KV_TOK if vbs else 0)
        order, batches = api.ss_schedule(cfg, g.prompt_len, g.pred_len)
        ocfg = osch.SchedCfg(use_vbs=vbs, kv_budget_bytes=cfg.kv_budget_bytes, kv_bytes_per_token=cfg.kv_bytes_per_token)
        _, ob = osch.plan(g.prompt_len, g.pred_len, ocfg)
        for n_gpus in (1, 2, 3, 8):
            got = api.ss_deal_batches(batches, order, g.prompt_len, W, KV_TOK, n_gpus)
            assert got == osch.deal(ob, g.prompt_len, W, KV_TOK, n_gpus)
            if n_gpus > 1:
                assert len(set(got)) == n_gpus


def _simulated_engine(g, cfg):
    """run_batches() of a rank without a GPU: the scheduler oracle's per-batch arithmetic."""
    def run(order, batches):
        n, mx = g.n, cfg.max_new_tokens
        tokens = np.zeros((n, mx), dtype=np.int32)
        lens, status = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.uint8)
        failed, log = [], []
        st = {"useful_tokens": 0, "row_steps": 0, "steps": 0, "kernel_launches": 0, "model_bytes": 0.0,
              "prefill_ms": 0.0, "decode_ms": 0.0}
        for first, rows, cap, rec in batches:
            ids = order[first:first + rows]
            steps = min(cap, max(int(g.true_len[r]) for r in ids))
            bad = [r for r in ids if int(g.true_len[r]) > cap and cap < mx]
            for r in ids:
                if r not in bad:
                    lens[r], status[r] = g.true_len[r], 1
                    tokens[r, :lens[r]] = r + 1
                    st["useful_tokens"] += int(lens[r])
            failed += bad
            log.append({"first_row": first, "n_rows": rows, "cap": cap, "is_recompute": rec, "steps": steps,
                        "n_failed": len(bad), "prefill_ms": 0.0, "decode_ms": float(steps)})
            st["steps"] += steps
            st["row_steps"] += rows * steps
            st["decode_ms"] += float(steps)
        return {"tokens": tokens, "len": lens, "status": status, "failed": failed, "log": log, "stats": st}
    return run


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2305_13144_b200 import api
    from paper_2305_13144_b200.replicas import run_group_replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def gather(obj):
        box = [None] * world
        dist.all_gather_object(box, obj)
        return box

    g = synth.group_7b_1024(seed=2)
    cfg = api.sched_cfg(use_vbs=True, kv_budget_bytes=int(120e9), kv_bytes_per_token=KV_TOK)
    res = run_group_replicas(api, cfg, g, None, rank=rank, world=world, run_batches=_simulated_engine(g, cfg),
                             gather=gather, shape=synth.LLAMA_7B)
    out.put((rank, res["order"].tolist(), res["failures"], res["len"].tolist(), res["status"].tolist(),
             [(b["first_row"], b["n_rows"], b["cap"], b["is_recompute"], b["steps"], b["n_failed"], b["gpu"])
              for b in res["log"]], res["stats"], res["device_s"], int(res["tokens"][:, 0].sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_serve_every_row_once_and_reproduce_the_single_gpu_log():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29741, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1:] == res[1][1:]                         # both ranks assembled the same result
    _, order, failures, lens, status, log, stats, device_s, tok0 = res[0]
    g = synth.group_7b_1024(seed=2)
    ocfg = osch.SchedCfg(use_vbs=True, kv_budget_bytes=int(120e9), kv_bytes_per_token=KV_TOK)
    sim = osch.simulate(g.prompt_len, g.pred_len, g.true_len, ocfg)
    n, nf = g.n, len(sim["failures"])
    assert order[:n] == sim["order"] and order[n:n + nf] == sim["failures"] and failures == sim["failures"]
    assert lens == g.true_len.tolist() and status == [1] * n            # every row served, to its end
    assert tok0 == sum(r + 1 for r in range(n))                          # ... exactly once, by whoever ran it
    assert len(log) == len(sim["batches"])
    for rec, ob in zip(log, sim["batches"]):                             # the single-GPU log, batch by batch
        assert order[rec[0]:rec[0] + rec[1]] == ob.rows
        assert rec[2:6] == (ob.cap, int(ob.is_recompute), ob.steps, len(ob.failed))
    assert {rec[6] for rec in log} == {0, 1}                             # both replicas worked
    assert stats["useful_tokens"] == sim["useful_tokens"] and stats["row_steps"] == sim["row_steps"]
    assert stats["steps"] == sim["steps"] and stats["n_failed"] == nf
    assert max(device_s) < 0.62 * sum(device_s)                          # longest-cost-first keeps the halves close
