"""CPU oracle for the sequence scheduler.  TEST INFRASTRUCTURE ONLY.

Plain Python, integer arithmetic, one function per rule of Sec. 4.1 of the paper, in the
paper's order: sort the group by predicted length and split it into micro-batches;
binning (cell 50, round up); failure collection and recomputation (FCR: cap the new
tokens of a batch at its largest predicted length, collect the rows that did not
finish, regenerate them at the end of the group); variable batch size (VBS: about the
same number of tokens per batch, 16 for L >= 300 and 256*50/L rounded to the nearest
power of two below that, Sec. 4.2 "Experimental Setting"); and the vanilla arm (fixed
batch, no scheduling).  Only tests, the smoke check and the benchmark's CPU-baseline
leg may use this file; it imports nothing from the CUDA package.

Readings taken where the paper is silent or garbled (each is also listed in the design
notes of the repository):
  * the VBS formula is printed as B0*L/L0, but the paragraph around it (Sec. 4.1, Variable Batch
    Size: shorter responses get bigger batches so that every batch holds about as many tokens)
    and the constants of the experiments (256*50/L, Sec. 4.2) fix B = B0*L0/L;
  * an exact multiple of the cell stays in its cell (100 -> 100); predictions < 1 clamp to 1;
  * the power of two nearest to 256*50/L (Sec. 4.2) is taken by linear distance, a tie goes down;
  * the threshold rule wins over the formula at L >= 300 (batch 16 although 12800/300 = 42.7);
  * a batch may straddle bins; the allowance of its longest (latest) row governs its size;
  * the sort is ascending and stable in the original index;
  * the cap counts the token produced by the prompt pass; a row whose length equals the
    cap has finished (its EOS is its cap-th token); one more is a failure;
  * a failed row's partial output is thrown away and the row is regenerated from its prompt,
    in batches of B0 in collection order with cap = max_new (so it cannot fail twice);
  * a key/value memory budget, if given, is one more admission test during batch formation,
    with the worst case (longest prompt so far + cap of the newest row) charged per row;
  * the vanilla order is a permutation passed in by the caller.

Parity status: pinned by tests/test_oracle_scheduler.py (the paper's VBS constants, two
hand-worked groups stored in tests/golden, edge cases and invariants).
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class SchedCfg:
    bin_size: int = 50            # 1 = no binning
    base_batch: int = 16          # B0
    use_vbs: bool = False
    use_fcr: bool = True
    vbs_len_threshold: int = 300
    vbs_token_budget: int = 256 * 50
    min_batch: int = 16
    max_batch: int = 256
    max_new_tokens: int = 512
    kv_budget_bytes: int = 0      # 0 = unlimited
    kv_bytes_per_token: int = 0
    vanilla: bool = False


@dataclass
class Batch:
    rows: list                    # original query ids, in order
    cap: int
    is_recompute: bool = False
    # filled by simulate():
    steps: int = 0
    failed: list = field(default_factory=list)


def bin_of(x: int, cfg: SchedCfg) -> int:
    """Round a length up to its cell (Sec. 4.1, Binning: a length goes to the closest cell boundary at
    or above it)."""
    x = min(max(int(x), 1), cfg.max_new_tokens)
    if cfg.bin_size == 1:
        return x
    return -(-x // cfg.bin_size) * cfg.bin_size


def round_pow2(num: int, den: int) -> int:
    """Nearest power of two to num/den (>= 1), linear distance, tie -> lower.  Exact in integers."""
    lo = 1
    while 2 * lo * den <= num:
        lo *= 2
    hi = 2 * lo
    # (num/den - lo) <= (hi - num/den)
    return lo if (num - lo * den) <= (hi * den - num) else hi


def vbs_batch(L: int, cfg: SchedCfg) -> int:
    """Batch size allowed for (binned) length L."""
    if not cfg.use_vbs:
        return cfg.base_batch
    if L >= cfg.vbs_len_threshold:
        return cfg.base_batch
    b = round_pow2(cfg.vbs_token_budget, L)
    return min(max(b, cfg.min_batch), cfg.max_batch)


def plan(prompt_len, pred_len, cfg: SchedCfg, perm=None):
    """First-pass plan: (order, batches).  `order` lists query ids in processing order;
    each Batch holds its slice of it."""
    n = len(pred_len)
    if cfg.vanilla:
        order = list(range(n)) if perm is None else [int(p) for p in perm]
        assert sorted(order) == list(range(n))
        batches = [Batch(order[i:i + cfg.base_batch], cfg.max_new_tokens)
                   for i in range(0, n, cfg.base_batch)]
        return order, batches

    bins = [bin_of(pred_len[i], cfg) for i in range(n)]
    order = sorted(range(n), key=lambda i: (bins[i], i))
    batches = []
    i = 0
    while i < n:
        B = 0
        maxp = 0
        while i + B < n:
            j = order[i + B]
            cap_j = min(bins[j], cfg.max_new_tokens)
            if B + 1 > vbs_batch(bins[j], cfg):
                break
            if cfg.kv_budget_bytes > 0 and B >= 1:
                need = (B + 1) * (max(maxp, int(prompt_len[j])) + cap_j) * cfg.kv_bytes_per_token
                if need > cfg.kv_budget_bytes:
                    break
            B += 1
            maxp = max(maxp, int(prompt_len[j]))
        rows = order[i:i + B]
        cap = min(max(bins[r] for r in rows), cfg.max_new_tokens) if cfg.use_fcr else cfg.max_new_tokens
        batches.append(Batch(rows, cap))
        i += B
    return order, batches


def simulate(prompt_len, pred_len, true_len, cfg: SchedCfg, perm=None) -> dict:
    """Run the group with termination forced by true_len (which counts the EOS).

    Returns the full batch log (first pass, then recompute batches) and the statistics
    the paper reports: per-batch length, redundancy, failure ratio.
    """
    n = len(true_len)
    order, batches = plan(prompt_len, pred_len, cfg, perm)
    failures = []
    for b in batches:
        b.steps = min(b.cap, max(int(true_len[r]) for r in b.rows))
        b.failed = [r for r in b.rows if int(true_len[r]) > b.cap and b.cap < cfg.max_new_tokens]
        failures.extend(b.failed)
    recompute = []
    for i in range(0, len(failures), cfg.base_batch):
        rows = failures[i:i + cfg.base_batch]
        rb = Batch(rows, cfg.max_new_tokens, is_recompute=True)
        rb.steps = min(rb.cap, max(int(true_len[r]) for r in rows))
        recompute.append(rb)
    log = batches + recompute
    useful = sum(int(t) for t in true_len)
    rowsteps = sum(len(b.rows) * b.steps for b in log)
    steps = sum(b.steps for b in log)
    return {
        "order": order,
        "batches": log,
        "failures": failures,
        "useful_tokens": useful,
        "steps": steps,
        "row_steps": rowsteps,
        "redundancy": 1.0 - useful / rowsteps if rowsteps else 0.0,
        "avg_len": steps / len(log) if log else 0.0,
        "avg_len_weighted": rowsteps / sum(len(b.rows) for b in log) if log else 0.0,
        "failure_ratio": len(failures) / n if n else 0.0,
    }


def deal(batches, prompt_len, weight_bytes: int, kv_bytes_per_token: int, n_gpus: int) -> list:
    """Replica dispatch of a batch list (Sec. 1 proposes handing micro-batches of different perceived lengths
    to different GPUs; the rule itself is this build's): cost of a batch = cap * (weight_bytes +
    rows * (mean prompt + cap / 2) * kv_bytes_per_token), all in integers; batches in order of decreasing cost
    (ties: lower index) each go to the replica with the smallest total so far (ties: lowest replica).
    Returns the replica of every batch."""
    cost = []
    for b in batches:
        tokens2 = 2 * sum(int(prompt_len[r]) for r in b.rows) + len(b.rows) * b.cap
        cost.append(b.cap * (weight_bytes + tokens2 * kv_bytes_per_token // 2))
    load = [0] * n_gpus
    out = [0] * len(batches)
    for i in sorted(range(len(batches)), key=lambda i: (-cost[i], i)):
        g = min(range(n_gpus), key=lambda g: (load[g], g))
        out[i] = g
        load[g] += cost[i]
    return out
