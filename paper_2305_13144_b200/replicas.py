"""One group of queries on several GPUs, each holding a replica of the weights.

The paper proposes the extension in one paragraph (Sec. 1): micro-batches of different perceived lengths can be
handed to different GPUs.  Nothing crosses between GPUs while batches run -- a micro-batch is an independent unit --
so there is no collective on the data path: every rank computes the same schedule and the same deal (both pure host
functions of the library), runs its own share with ss_run_batches(), and the ranks exchange only small host-side
records (which rows failed, the batch log, the finished rows) through `gather`, normally
torch.distributed.all_gather_object.  The rows the caps cut are requeued exactly as on one GPU: collected in batch
and row order, cut into batches of B0 with cap = max_new, dealt again.

This module only sequences calls of the C ABI and moves host records; it computes nothing of the method.
"""
from __future__ import annotations

import numpy as np


def weight_bytes_per_step(shape) -> int:
    d, F, V, L = shape.d_model, shape.d_ffn, shape.vocab, shape.n_layers
    return L * (4 * d * d + 3 * d * F + 2 * d) * 2 + V * d * 2 + d * 2


def run_group_replicas(api, cfg, group, perm, *, rank: int, world: int, run_batches, gather, shape) -> dict:
    """Runs `group` on `world` replicas.  run_batches(order, batches) runs a batch list on this rank's engine and
    returns what api.ss_run_batches() returns; gather(obj) returns the list of every rank's obj, in rank order.
    Every rank returns the assembled result: order [2n], failures, log (first pass in batch order, then the
    recomputation), tokens / len / status over the group, and per-rank device seconds."""
    n = group.n
    kv_tok = 2 * shape.d_model * 2 * shape.n_layers
    W = weight_bytes_per_step(shape)
    order, batches = api.ss_schedule(cfg, group.prompt_len, group.pred_len, perm)
    order = order.tolist()
    mx = cfg.max_new_tokens
    tokens = np.zeros((n, mx), dtype=np.int32)
    lens = np.zeros(n, dtype=np.int32)
    status = np.zeros(n, dtype=np.uint8)
    log, device_ms = [], np.zeros(world)
    totals = {"useful_tokens": 0, "row_steps": 0, "steps": 0, "kernel_launches": 0, "model_bytes": 0.0}

    def one_pass(order_now, batch_list):
        """Deal, run this rank's share, exchange; returns the failures of the pass in batch and row order."""
        gpu_of = api.ss_deal_batches(batch_list, order_now, group.prompt_len, W, kv_tok, world)
        mine = [i for i, g in enumerate(gpu_of) if g == rank]
        res = run_batches(order_now, [batch_list[i] for i in mine])
        cut = set(res["failed"])
        done = [r for i in mine for r in order_now[batch_list[i][0]:batch_list[i][0] + batch_list[i][1]] if r not in cut]
        # failures per batch: ss_run_batches lists them in batch and row order; the log says how many each batch had
        per_batch, k = {}, 0
        for i, rec in zip(mine, res["log"]):
            per_batch[i] = res["failed"][k:k + rec["n_failed"]]
            k += rec["n_failed"]
        record = {"batches": mine, "log": res["log"], "failed": per_batch, "rows": done,
                  "len": res["len"][done].tolist(), "status": res["status"][done].tolist(),
                  "tokens": [res["tokens"][r, :res["len"][r]].tolist() for r in done],
                  "ms": res["stats"]["prefill_ms"] + res["stats"]["decode_ms"],
                  "stats": {k2: res["stats"][k2] for k2 in totals}}
        pass_log, failed = {}, {}
        for rk, rec in enumerate(gather(record)):
            device_ms[rk] += rec["ms"]
            for k2 in totals:
                totals[k2] += rec["stats"][k2]
            for i, lg in zip(rec["batches"], rec["log"]):
                pass_log[i] = dict(lg, gpu=rk)
            failed.update(rec["failed"])
            for r, ln, st, tk in zip(rec["rows"], rec["len"], rec["status"], rec["tokens"]):
                lens[r], status[r] = ln, st
                tokens[r, :ln] = tk
        log.extend(pass_log[i] for i in range(len(batch_list)))
        return [r for i in range(len(batch_list)) for r in failed.get(i, [])]

    failures = one_pass(order, batches)
    B0 = cfg.base_batch
    order2 = order + failures
    again = [(n + i, min(B0, len(failures) - i), mx, 1) for i in range(0, len(failures), B0)]
    if again:
        left = one_pass(order2, again)
        assert not left, "a row regenerated with cap = max_new cannot fail again"
    return {"order": np.array(order2 + [-1] * (n - len(failures)), dtype=np.int32), "failures": failures, "log": log,
            "tokens": tokens, "len": lens, "status": status, "device_s": (device_ms / 1e3).tolist(),
            "stats": dict(totals, n_failed=len(failures), n_batches=len(log))}
