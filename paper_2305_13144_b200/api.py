"""Thin ctypes binding of the C ABI in include/seqsched.h (same names, argument marshalling only).

Every step of the path runs inside libseqsched.so; nothing here computes.  Device buffers are
torch CUDA tensors (torch provides device memory and the stream), host buffers are numpy arrays.
If the shared library is missing or does not load, importing a symbol from here raises: there is
no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libseqsched.so")

SS_OK = 0
SS_ERR_ARG, SS_ERR_CAPACITY, SS_ERR_KV_BUDGET, SS_ERR_STATE = -1, -2, -3, -4
SS_ERR_CUDA, SS_ERR_DEVICE_TIMEOUT, SS_ERR_UNSUPPORTED = -5, -6, -7

EXPORTS = [
    "ss_arena_bytes", "ss_create", "ss_destroy", "ss_load_weights", "ss_schedule", "ss_prefill",
    "ss_decode_step", "ss_decode_steps", "ss_read_batch", "ss_release_batch", "ss_run_group",
    "ss_step_model_bytes", "ss_strerror", "ss_last_device_status", "ss_last_cuda_error", "ss_kernel_launches",
    "ss_logits_noalloc", "ss_step_trace", "ss_set_trace", "ss_set_sampling", "ss_set_row_keys", "ss_run_batches", "ss_deal_batches", "ss_keep_prompts", "ss_resume", "ss_drop_prompts",
    "ss_set_prompt_cache", "ss_set_wait_limit_ms", "ss_selftest_wait_timeout",
]


class SSError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ss_strerror(code)} ({code})")


class ss_model_cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab", "eos_id")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)]


class ss_runtime_cfg(C.Structure):
    _fields_ = [("max_batch", C.c_int32), ("max_ctx", C.c_int32), ("max_prefill_tokens", C.c_int32),
                ("max_new_tokens", C.c_int32), ("kv_pool_tokens", C.c_int64)]


class ss_sched_cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("bin_size", "base_batch", "use_vbs", "use_fcr", "vbs_len_threshold",
                                         "vbs_token_budget", "min_batch", "max_batch", "max_new_tokens", "vanilla")] + \
               [("kv_budget_bytes", C.c_int64), ("kv_bytes_per_token", C.c_int64)]


class ss_batch_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("first_row", "n_rows", "cap", "is_recompute")]


class ss_tensor_desc(C.Structure):
    _fields_ = [("name", C.c_char_p), ("data", C.c_void_p), ("is_device", C.c_int32),
                ("rows", C.c_int64), ("cols", C.c_int64)]


class ss_step_opts(C.Structure):
    _fields_ = [("forced_tokens", C.c_void_p), ("dump_logits", C.c_void_p), ("dump_hidden", C.c_void_p),
                ("dump_choice", C.c_void_p)]


class ss_batch_log(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("first_row", "n_rows", "cap", "is_recompute", "steps", "n_failed")] + \
               [("prefill_ms", C.c_float), ("decode_ms", C.c_float)]


class ss_group_stats(C.Structure):
    _fields_ = [("useful_tokens", C.c_int64), ("row_steps", C.c_int64), ("steps", C.c_int64),
                ("n_batches", C.c_int32), ("n_failed", C.c_int32),
                ("total_ms", C.c_float), ("prefill_ms", C.c_float), ("decode_ms", C.c_float),
                ("model_bytes", C.c_double), ("kernel_launches", C.c_int64)]


_lib_handle = None


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2305_13144_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.ss_strerror.restype = C.c_char_p
        L.ss_strerror.argtypes = [C.c_int]
        L.ss_kernel_launches.restype = C.c_int64
        L.ss_kernel_launches.argtypes = [C.c_void_p]
        L.ss_last_cuda_error.argtypes = [C.c_void_p]
        L.ss_arena_bytes.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_size_t)]
        L.ss_create.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
        L.ss_destroy.argtypes = [C.c_void_p]
        L.ss_load_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.ss_schedule.argtypes = [C.c_void_p] * 4 + [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.ss_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32,
                                 C.c_void_p, C.c_void_p]
        L.ss_decode_step.argtypes = [C.c_void_p] * 4
        L.ss_decode_steps.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.ss_read_batch.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.ss_release_batch.argtypes = [C.c_void_p]
        L.ss_run_group.argtypes = [C.c_void_p] * 7 + [C.c_int32] + [C.c_void_p] * 6 + [C.c_int32, C.c_void_p, C.c_void_p]
        L.ss_run_batches.argtypes = [C.c_void_p] * 5 + [C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32] + \
                                    [C.c_void_p] * 6 + [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.ss_deal_batches.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32,
                                      C.c_void_p]
        L.ss_keep_prompts.argtypes = [C.c_void_p] * 3
        L.ss_resume.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.ss_drop_prompts.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.ss_set_prompt_cache.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32]
        L.ss_step_model_bytes.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_double)]
        L.ss_last_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_uint32)]
        L.ss_step_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        L.ss_set_trace.argtypes = [C.c_void_p, C.c_int32]
        L.ss_set_wait_limit_ms.argtypes = [C.c_void_p, C.c_int32]
        L.ss_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_int32]
        L.ss_set_sampling.argtypes = [C.c_void_p, C.c_float, C.c_uint64]
        L.ss_set_row_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.ss_logits_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_float, C.c_void_p, C.c_void_p]
        _lib_handle = L
    return _lib_handle


def ss_strerror(code: int) -> str:
    return lib().ss_strerror(int(code)).decode()


def _check(code: int, where: str, ctx=None) -> None:
    if code != SS_OK:
        if code == SS_ERR_CUDA and ctx is not None and ctx.handle:
            where += f" [cuda error {lib().ss_last_cuda_error(ctx.handle)}]"
        raise SSError(code, where)


def _np(a, dtype):
    if a is None:
        return None
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def _hp(a):
    """Pointer of a host numpy array (or None)."""
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dp(t):
    """Pointer of a device tensor (or None).  Host tensors are rejected."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def model_cfg(shape) -> ss_model_cfg:
    return ss_model_cfg(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                        shape.eos_id, shape.rms_eps, shape.rope_theta)


def sched_cfg(*, bin_size=50, base_batch=16, use_vbs=False, use_fcr=True, vbs_len_threshold=300,
              vbs_token_budget=256 * 50, min_batch=16, max_batch=256, max_new_tokens=512, vanilla=False,
              kv_budget_bytes=0, kv_bytes_per_token=0) -> ss_sched_cfg:
    return ss_sched_cfg(bin_size, base_batch, int(use_vbs), int(use_fcr), vbs_len_threshold, vbs_token_budget,
                        min_batch, max_batch, max_new_tokens, int(vanilla), kv_budget_bytes, kv_bytes_per_token)


def ss_arena_bytes(model: ss_model_cfg, rt: ss_runtime_cfg) -> int:
    out = C.c_size_t(0)
    _check(lib().ss_arena_bytes(C.byref(model), C.byref(rt), C.byref(out)), "ss_arena_bytes")
    return out.value


class Ctx:
    """Opaque ss_ctx* plus references that must outlive it (arena, stream)."""

    def __init__(self, handle, arena, stream, model, rt):
        self.handle, self.arena, self.stream, self.model, self.rt = handle, arena, stream, model, rt

    def __del__(self):
        try:
            if self.handle:
                lib().ss_destroy(self.handle)
                self.handle = None
        except Exception:
            pass


def ss_create(model: ss_model_cfg, rt: ss_runtime_cfg, arena, stream=None) -> Ctx:
    """arena: uint8 CUDA tensor of at least ss_arena_bytes(); stream: torch.cuda.Stream or None (current)."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    off = (-arena.data_ptr()) % 1024
    h = C.c_void_p()
    _check(lib().ss_create(C.byref(model), C.byref(rt), C.c_void_p(arena.data_ptr() + off), arena.numel() - off,
                           C.c_void_p(stream.cuda_stream), C.byref(h)), "ss_create")
    return Ctx(h, arena, stream, model, rt)


def ss_destroy(ctx: Ctx) -> None:
    if ctx.handle:
        _check(lib().ss_destroy(ctx.handle), "ss_destroy")
        ctx.handle = None


def ss_load_weights(ctx: Ctx, tensors: dict) -> None:
    """tensors: name -> bf16 CUDA tensor, or numpy uint16 array of bf16 bit patterns (host)."""
    descs = (ss_tensor_desc * len(tensors))()
    keep = []
    if any(not isinstance(t, np.ndarray) and t.is_cuda for t in tensors.values()):
        # device tensors are usually produced on torch's current stream; the engine reads them on its own
        import torch
        torch.cuda.current_stream().synchronize()
    for i, (name, t) in enumerate(tensors.items()):
        if isinstance(t, np.ndarray):
            a = np.ascontiguousarray(t, dtype=np.uint16)
            keep.append(a)
            ptr, dev, shape = a.ctypes.data, 0, a.shape
        else:
            if not t.is_contiguous() or t.element_size() != 2:
                raise ValueError(f"{name}: expected contiguous bf16")
            keep.append(t)
            ptr, dev, shape = t.data_ptr(), int(t.is_cuda), tuple(t.shape)
        rows, cols = (1, shape[0]) if len(shape) == 1 else shape
        descs[i] = ss_tensor_desc(name.encode(), ptr, dev, rows, cols)
    _check(lib().ss_load_weights(ctx.handle, descs, len(tensors)), "ss_load_weights", ctx)


def ss_schedule(cfg: ss_sched_cfg, prompt_len, pred_len, perm=None):
    """Returns (order int32 [n], list of (first_row, n_rows, cap, is_recompute))."""
    pl, pr, pm = _np(prompt_len, np.int32), _np(pred_len, np.int32), _np(perm, np.int32)
    n = int(pr.shape[0])
    order = np.zeros(max(n, 1), dtype=np.int32)
    cap = max(n, 1)
    batches = (ss_batch_desc * cap)()
    nb = C.c_int32(0)
    _check(lib().ss_schedule(C.byref(cfg), _hp(pl), _hp(pr), _hp(pm), n, _hp(order), batches, cap, C.byref(nb)),
           "ss_schedule")
    return order[:n], [(b.first_row, b.n_rows, b.cap, b.is_recompute) for b in batches[:nb.value]]


def _opts(forced_tokens=None, dump_logits=None, dump_hidden=None, dump_choice=None):
    if forced_tokens is None and dump_logits is None and dump_hidden is None and dump_choice is None:
        return None
    return ss_step_opts(_dp(forced_tokens), _dp(dump_logits), _dp(dump_hidden), _dp(dump_choice))


def ss_prefill(ctx: Ctx, tokens, cu_seqlens, eos_at, cap: int, *, forced_tokens=None, dump_logits=None,
               dump_hidden=None, dump_choice=None, first_tokens=None) -> None:
    tk, cu, ea = _np(tokens, np.int32), _np(cu_seqlens, np.int32), _np(eos_at, np.int32)
    o = _opts(forced_tokens, dump_logits, dump_hidden, dump_choice)
    _check(lib().ss_prefill(ctx.handle, _hp(tk), _hp(cu), int(cu.shape[0]) - 1, _hp(ea), int(cap),
                            C.byref(o) if o else None, _dp(first_tokens)), "ss_prefill", ctx)


def ss_keep_prompts(ctx: Ctx, ids, keep_len) -> None:
    i, k = _np(ids, np.int32), _np(keep_len, np.int32)
    _check(lib().ss_keep_prompts(ctx.handle, _hp(i), _hp(k)), "ss_keep_prompts", ctx)


def ss_resume(ctx: Ctx, ids, eos_at, cap: int, *, forced_tokens=None, dump_logits=None, dump_hidden=None,
              dump_choice=None, first_tokens=None) -> None:
    i, ea = _np(ids, np.int32), _np(eos_at, np.int32)
    o = _opts(forced_tokens, dump_logits, dump_hidden, dump_choice)
    _check(lib().ss_resume(ctx.handle, _hp(i), int(i.shape[0]), _hp(ea), int(cap), C.byref(o) if o else None,
                           _dp(first_tokens)), "ss_resume", ctx)


def ss_drop_prompts(ctx: Ctx, ids=None) -> None:
    if ids is None:
        _check(lib().ss_drop_prompts(ctx.handle, None, -1), "ss_drop_prompts", ctx)
    else:
        i = _np(ids, np.int32)
        _check(lib().ss_drop_prompts(ctx.handle, _hp(i), int(i.shape[0])), "ss_drop_prompts", ctx)


def ss_set_prompt_cache(ctx: Ctx, mode: int, keep_len=None) -> None:
    k = _np(keep_len, np.int32)
    _check(lib().ss_set_prompt_cache(ctx.handle, int(mode), _hp(k), 0 if k is None else int(k.shape[0])),
           "ss_set_prompt_cache", ctx)


def ss_decode_step(ctx: Ctx, *, forced_tokens=None, dump_logits=None, dump_hidden=None, dump_choice=None,
                   next_tokens=None, n_active_host=None) -> None:
    """n_active_host: pinned int32 torch tensor (host) or None."""
    o = _opts(forced_tokens, dump_logits, dump_hidden, dump_choice)
    nah = None if n_active_host is None else C.c_void_p(n_active_host.data_ptr())
    _check(lib().ss_decode_step(ctx.handle, C.byref(o) if o else None, _dp(next_tokens), nah), "ss_decode_step", ctx)


def ss_decode_steps(ctx: Ctx, n_steps: int, n_active_host=None) -> None:
    nah = None if n_active_host is None else C.c_void_p(n_active_host.data_ptr())
    _check(lib().ss_decode_steps(ctx.handle, int(n_steps), nah), "ss_decode_steps", ctx)


def ss_read_batch(ctx: Ctx, B: int, stride: int):
    toks = np.zeros((B, stride), dtype=np.int32)
    lens = np.zeros(B, dtype=np.int32)
    status = np.zeros(B, dtype=np.uint8)
    _check(lib().ss_read_batch(ctx.handle, _hp(toks), stride, _hp(lens), _hp(status)), "ss_read_batch", ctx)
    return toks, lens, status


def ss_release_batch(ctx: Ctx) -> None:
    _check(lib().ss_release_batch(ctx.handle), "ss_release_batch", ctx)


def ss_run_group(ctx: Ctx, cfg: ss_sched_cfg, prompt_tokens, prompt_off, pred_len, perm=None, eos_at=None) -> dict:
    pt, po = _np(prompt_tokens, np.int32), _np(prompt_off, np.int64)
    pr, pm, ea = _np(pred_len, np.int32), _np(perm, np.int32), _np(eos_at, np.int32)
    n = int(pr.shape[0])
    mx = cfg.max_new_tokens
    out_off = np.arange(n + 1, dtype=np.int64) * mx
    out_tokens = np.zeros(max(n * mx, 1), dtype=np.int32)
    out_len = np.zeros(max(n, 1), dtype=np.int32)
    out_status = np.zeros(max(n, 1), dtype=np.uint8)
    order = np.full(max(2 * n, 1), -1, dtype=np.int32)
    log_cap = 2 * n + 2
    log = (ss_batch_log * log_cap)()
    n_log = C.c_int32(0)
    stats = ss_group_stats()
    _check(lib().ss_run_group(ctx.handle, C.byref(cfg), _hp(pt), _hp(po), _hp(pr), _hp(pm), _hp(ea), n,
                              _hp(out_tokens), _hp(out_off), _hp(out_len), _hp(out_status), _hp(order),
                              log, log_cap, C.byref(n_log), C.byref(stats)), "ss_run_group", ctx)
    fields = [f[0] for f in ss_batch_log._fields_]
    return {
        "tokens": out_tokens.reshape(n, mx) if n else out_tokens[:0].reshape(0, mx),
        "len": out_len[:n], "status": out_status[:n], "order": order[:2 * n],
        "log": [{f: getattr(b, f) for f in fields} for b in log[:n_log.value]],
        "stats": {f[0]: getattr(stats, f[0]) for f in ss_group_stats._fields_},
    }


def _descs(batches):
    arr = (ss_batch_desc * max(len(batches), 1))()
    for i, b in enumerate(batches):
        arr[i] = ss_batch_desc(*[int(x) for x in b])
    return arr


def ss_run_batches(ctx: Ctx, cfg: ss_sched_cfg, prompt_tokens, prompt_off, eos_at, order, batches) -> dict:
    """batches: list of (first_row, n_rows, cap, is_recompute) indexing `order`.  Returns tokens / len / status
    arrays over the whole group (valid for the rows that ended here), the failed queries, the log and the stats."""
    pt, po, ea = _np(prompt_tokens, np.int32), _np(prompt_off, np.int64), _np(eos_at, np.int32)
    od = _np(order, np.int32)
    n = int(po.shape[0]) - 1
    mx = cfg.max_new_tokens
    out_off = np.arange(n + 1, dtype=np.int64) * mx
    out_tokens = np.zeros(max(n * mx, 1), dtype=np.int32)
    out_len = np.zeros(max(n, 1), dtype=np.int32)
    out_status = np.zeros(max(n, 1), dtype=np.uint8)
    fail = np.zeros(max(n, 1), dtype=np.int32)
    n_fail, n_log = C.c_int32(0), C.c_int32(0)
    log = (ss_batch_log * max(len(batches), 1))()
    stats = ss_group_stats()
    _check(lib().ss_run_batches(ctx.handle, C.byref(cfg), _hp(pt), _hp(po), _hp(ea), n, _hp(od), int(od.shape[0]),
                                _descs(batches), len(batches), _hp(out_tokens), _hp(out_off), _hp(out_len),
                                _hp(out_status), _hp(fail), C.byref(n_fail), log, len(batches), C.byref(n_log),
                                C.byref(stats)), "ss_run_batches", ctx)
    fields = [f[0] for f in ss_batch_log._fields_]
    return {"tokens": out_tokens.reshape(n, mx), "len": out_len[:n], "status": out_status[:n],
            "failed": fail[:n_fail.value].tolist(),
            "log": [{f: getattr(b, f) for f in fields} for b in log[:n_log.value]],
            "stats": {f[0]: getattr(stats, f[0]) for f in ss_group_stats._fields_}}


def ss_deal_batches(batches, order, prompt_len, weight_bytes: int, kv_bytes_per_token: int, n_gpus: int) -> list:
    od, pl = _np(order, np.int32), _np(prompt_len, np.int32)
    out = np.zeros(max(len(batches), 1), dtype=np.int32)
    _check(lib().ss_deal_batches(_descs(batches), len(batches), _hp(od), _hp(pl), int(weight_bytes),
                                 int(kv_bytes_per_token), int(n_gpus), _hp(out)), "ss_deal_batches")
    return out[:len(batches)].tolist()


def ss_step_model_bytes(ctx: Ctx, ctx_len, active=None) -> float:
    cl, ac = _np(ctx_len, np.int32), _np(active, np.uint8)
    out = C.c_double(0)
    _check(lib().ss_step_model_bytes(ctx.handle, _hp(cl), _hp(ac), int(cl.shape[0]), C.byref(out)),
           "ss_step_model_bytes")
    return out.value


def ss_last_device_status(ctx: Ctx) -> int:
    out = C.c_uint32(0)
    _check(lib().ss_last_device_status(ctx.handle, C.byref(out)), "ss_last_device_status", ctx)
    return out.value


def ss_set_sampling(ctx: Ctx, temperature: float, seed: int = 0) -> None:
    _check(lib().ss_set_sampling(ctx.handle, float(temperature), int(seed)), "ss_set_sampling", ctx)


def ss_set_row_keys(ctx: Ctx, keys) -> None:
    k = _np(keys, np.int32)
    _check(lib().ss_set_row_keys(ctx.handle, _hp(k), int(k.shape[0])), "ss_set_row_keys", ctx)


def ss_set_wait_limit_ms(ctx: Ctx, ms: int) -> None:
    _check(lib().ss_set_wait_limit_ms(ctx.handle, int(ms)), "ss_set_wait_limit_ms", ctx)


def ss_selftest_wait_timeout(ctx: Ctx, limit_us: int) -> int:
    """Returns the code the runtime reports after a wait that cannot complete (SS_ERR_DEVICE_TIMEOUT)."""
    return int(lib().ss_selftest_wait_timeout(ctx.handle, int(limit_us)))


def ss_set_trace(ctx: Ctx, on: bool) -> None:
    _check(lib().ss_set_trace(ctx.handle, int(bool(on))), "ss_set_trace", ctx)


def ss_step_trace(ctx: Ctx) -> np.ndarray:
    """Stage-boundary time stamps (ns) of the last decode step, see include/seqsched.h."""
    n = C.c_int32(0)
    cap = 2 + 4 * (4 * ctx.model.n_layers + 1)
    out = np.zeros(cap, dtype=np.uint64)
    _check(lib().ss_step_trace(ctx.handle, _hp(out), cap, C.byref(n)), "ss_step_trace", ctx)
    return out[:n.value]


def ss_last_cuda_error(ctx: Ctx) -> int:
    return lib().ss_last_cuda_error(ctx.handle)


def ss_kernel_launches(ctx: Ctx) -> int:
    return lib().ss_kernel_launches(ctx.handle)


def ss_logits_noalloc(hidden, norm_gain, lm_head, rms_eps: float, logits, stream=None) -> None:
    """LM-head logits without any allocation by the library (see include/seqsched.h).

    hidden fp32 [n, d], norm_gain bf16 [d], lm_head bf16 [V, d], logits fp32 [n, V]: CUDA tensors
    the caller made beforehand.  Scratch comes from a fixed array inside the library, shared by
    all calls: keep the calls of one device in one stream order."""
    import torch
    n, d = hidden.shape
    V = lm_head.shape[0]
    if hidden.dtype != torch.float32 or logits.dtype != torch.float32 or tuple(logits.shape) != (n, V):
        raise ValueError("hidden and logits must be fp32 [n, d] / [n, V]")
    if norm_gain.element_size() != 2 or lm_head.element_size() != 2:
        raise ValueError("norm_gain and lm_head must be bf16")
    st = torch.cuda.current_stream() if stream is None else stream
    _check(lib().ss_logits_noalloc(_dp(hidden), _dp(norm_gain), _dp(lm_head), n, d, V, float(rms_eps), _dp(logits),
                                   C.c_void_p(st.cuda_stream)), "ss_logits_noalloc")


def runtime_cfg(max_batch, max_ctx, max_prefill_tokens, max_new_tokens, kv_pool_tokens) -> ss_runtime_cfg:
    return ss_runtime_cfg(max_batch, max_ctx, max_prefill_tokens, max_new_tokens, kv_pool_tokens)


def make_engine(shape, rt: ss_runtime_cfg, weights: dict, device="cuda:0") -> Ctx:
    """Convenience for tests and the benchmark: allocate the arena with torch, create, load weights.

    The engine gets a stream of its own; callers order their own work against it with
    torch.cuda.synchronize() or stream events."""
    import torch
    m = model_cfg(shape)
    nbytes = ss_arena_bytes(m, rt)
    with torch.cuda.device(device):
        arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        torch.cuda.synchronize()
        ctx = ss_create(m, rt, arena, torch.cuda.Stream())
        ss_load_weights(ctx, weights)
    return ctx
