"""CPU oracle for the decoder half of the hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow numpy implementation of what batched greedy decoding of a
LLaMA-style pre-norm decoder computes.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may use it; the product path never does, and this
file imports nothing from the CUDA package.

The paper (Sec. 4.1; App. D) treats the model as a given "LLaMA-based" decoder and
prints no equations for it, so the definition written out here is the textbook one.
Every constant the paper leaves open is an explicit argument:

    h0 = E[tok]
    per layer:  u  = RMSNorm(h; g_attn)            u_i = h_i * (mean_j h_j^2 + eps)^-1/2 * g_i
                q,k,v = Wq u, Wk u, Wv u           (no bias), split into H heads of Dh
                q,k <- RoPE(q or k, position)      rotate-half pairing (i, i + Dh/2),
                                                   angle = pos * theta^(-2i/Dh)
                o_h = sum_{j<=p} softmax_j(q_h . k_jh / sqrt(Dh)) v_jh       (causal, full MHA)
                h  <- h + Wo concat_h(o_h)
                u2 = RMSNorm(h; g_ffn)
                h  <- h + Wd ( silu(Wg u2) * (Wu u2) ),   silu(x) = x / (1 + exp(-x))
    logits = Wlm RMSNorm(h_L; g_final);  next token = argmax (lowest id wins a tie)

Three routes through the same definition are kept on purpose, because their
agreement is one of the pins: full recomputation over the whole prefix
(`forward_full`), incremental decoding with a KV cache (`KVDecoder`) and a
left-padded rectangular batch with an additive mask (`forward_padded`).

Precision: `dtype` (default float64).  Weights are whatever values the caller
passes (the tests pass bf16-representable values).

Parity status: every operator and the composition are pinned by tests/test_oracle_decoder.py
(closed forms, hand-worked values in tests/golden, brute force on tiny inputs and the
three-route invariants).  The absolute logits of a random model are pinned only through
that chain.
"""
from __future__ import annotations

import math
import numpy as np

from .sampler import sample_token


# ----------------------------------------------------------------------------- operators

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y_i = x_i / sqrt(mean_j x_j^2 + eps) * g_i over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding on the last axis (size Dh, even).

    x: [..., Dh]; pos: integer array broadcastable to x.shape[:-1].
    Pair (i, i + Dh/2) is rotated by the angle pos * theta^(-2i/Dh):
        x_i'        = x_i cos - x_{i+Dh/2} sin
        x_{i+Dh/2}' = x_{i+Dh/2} cos + x_i sin
    """
    dh = x.shape[-1]
    half = dh // 2
    i = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / dh)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c = np.cos(ang).astype(x.dtype)
    s = np.sin(ang).astype(x.dtype)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def softmax_attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, bias: np.ndarray | None = None) -> np.ndarray:
    """One query against n keys: sum_j softmax_j(q.k_j / sqrt(Dh) + bias_j) v_j.

    q: [Dh]; K, V: [n, Dh]; bias: [n] additive (0 or -inf), optional.
    """
    s = K @ q / math.sqrt(q.shape[-1])
    if bias is not None:
        s = s + bias
    s = s - np.max(s)
    p = np.exp(s)
    p = p / np.sum(p)
    return p @ V


def select_token(logits: np.ndarray, eos_id: int, suppress_eos: bool) -> int:
    """Greedy choice: the largest logit, lowest id on ties; EOS left out when suppressed."""
    if np.isnan(logits).any():
        raise FloatingPointError("NaN logit")
    l = logits
    if suppress_eos:
        l = logits.copy()
        l[eos_id] = -np.inf
    return int(np.argmax(l))          # numpy returns the first maximal index


# ----------------------------------------------------------------------------- the model

class Decoder:
    """Holds weights (dict of arrays, projection matrices [out, in]) and hyper-parameters."""

    def __init__(self, weights: dict, *, n_layers: int, n_heads: int, head_dim: int,
                 rms_eps: float = 1e-6, rope_theta: float = 10000.0, eos_id: int = 2,
                 dtype=np.float64):
        self.L, self.H, self.Dh = n_layers, n_heads, head_dim
        self.eps, self.theta, self.eos_id = rms_eps, rope_theta, eos_id
        self.dtype = np.dtype(dtype)
        self.w = {k: np.asarray(v, dtype=self.dtype) for k, v in weights.items()}
        self.d = self.w["embed"].shape[1]
        assert self.H * self.Dh == self.d

    # -- pieces shared by the three routes (each is one line of the definition) --
    def _qkv(self, l: int, h: np.ndarray, pos: np.ndarray):
        """h [T,d], pos [T] -> q,k,v [T,H,Dh] with RoPE applied to q and k."""
        w = self.w
        u = rmsnorm(h, w[f"l{l}.attn_norm"], self.eps)
        T = h.shape[0]
        q = (u @ w[f"l{l}.wq"].T).reshape(T, self.H, self.Dh)
        k = (u @ w[f"l{l}.wk"].T).reshape(T, self.H, self.Dh)
        v = (u @ w[f"l{l}.wv"].T).reshape(T, self.H, self.Dh)
        q = rope(q, pos[:, None], self.theta)
        k = rope(k, pos[:, None], self.theta)
        return q, k, v

    def _ffn(self, l: int, h: np.ndarray) -> np.ndarray:
        w = self.w
        u2 = rmsnorm(h, w[f"l{l}.ffn_norm"], self.eps)
        a = silu(u2 @ w[f"l{l}.w_gate"].T) * (u2 @ w[f"l{l}.w_up"].T)
        return h + a @ w[f"l{l}.w_down"].T

    def logits_of(self, h: np.ndarray) -> np.ndarray:
        return rmsnorm(h, self.w["final_norm"], self.eps) @ self.w["lm_head"].T

    # -- route 1: recompute the whole prefix ------------------------------------------
    def forward_full(self, tokens) -> tuple[np.ndarray, np.ndarray]:
        """tokens [T] -> (final hidden [T,d] before the last norm, logits [T,V])."""
        tokens = np.asarray(tokens, dtype=np.int64)
        T = tokens.shape[0]
        pos = np.arange(T)
        h = self.w["embed"][tokens].copy()
        for l in range(self.L):
            q, k, v = self._qkv(l, h, pos)
            o = np.zeros((T, self.H, self.Dh), dtype=self.dtype)
            for t in range(T):
                for hd in range(self.H):
                    o[t, hd] = softmax_attend(q[t, hd], k[:t + 1, hd], v[:t + 1, hd])
            h = h + o.reshape(T, self.d) @ self.w[f"l{l}.wo"].T
            h = self._ffn(l, h)
        return h, self.logits_of(h)

    # -- route 3: left-padded rectangle with an additive mask -----------------------------
    def forward_padded(self, seqs: list) -> tuple[np.ndarray, np.ndarray]:
        """Rows of unequal length, left-padded with token 0 to the longest.

        Returns (hidden [B,d], logits [B,V]) of each row's LAST position.  Pad keys are
        masked with -inf; a pad query sees only itself (its output is never used).
        Positions count from each row's first real token.
        """
        B = len(seqs)
        S = max(len(s) for s in seqs)
        pad = np.array([S - len(s) for s in seqs])
        tok = np.zeros((B, S), dtype=np.int64)
        for b, s in enumerate(seqs):
            tok[b, pad[b]:] = np.asarray(s)
        idx = np.arange(S)
        pos = np.maximum(idx[None, :] - pad[:, None], 0)                     # [B,S]
        real = idx[None, :] >= pad[:, None]                                   # [B,S]
        # bias[b, query, key]
        allowed = (idx[None, None, :] <= idx[None, :, None]) & real[:, None, :] & real[:, :, None]
        allowed |= np.eye(S, dtype=bool)[None]
        bias = np.where(allowed, 0.0, -np.inf).astype(self.dtype)
        h = self.w["embed"][tok].copy()                                       # [B,S,d]
        for l in range(self.L):
            hb = np.empty_like(h)
            for b in range(B):
                q, k, v = self._qkv(l, h[b], pos[b])
                o = np.zeros((S, self.H, self.Dh), dtype=self.dtype)
                for t in range(S):
                    for hd in range(self.H):
                        o[t, hd] = softmax_attend(q[t, hd], k[:, hd], v[:, hd], bias[b, t])
                hb[b] = h[b] + o.reshape(S, self.d) @ self.w[f"l{l}.wo"].T
            h = self._ffn(l, hb)
        last = h[:, -1, :]
        return last, self.logits_of(last)


class KVDecoder:
    """Route 2: incremental decoding of ONE sequence with a key/value cache."""

    def __init__(self, model: Decoder):
        self.m = model
        self.K = [np.zeros((0, model.H, model.Dh), dtype=model.dtype) for _ in range(model.L)]
        self.V = [np.zeros((0, model.H, model.Dh), dtype=model.dtype) for _ in range(model.L)]
        self.n = 0                      # tokens in the cache

    def feed(self, tokens) -> tuple[np.ndarray, np.ndarray]:
        """Append tokens (a prompt, or one generated token); returns (hidden [d], logits [V])
        of the last token fed."""
        m = self.m
        tokens = np.atleast_1d(np.asarray(tokens, dtype=np.int64))
        T = tokens.shape[0]
        pos = self.n + np.arange(T)
        h = m.w["embed"][tokens].copy()
        for l in range(m.L):
            q, k, v = m._qkv(l, h, pos)
            self.K[l] = np.concatenate([self.K[l], k], axis=0)
            self.V[l] = np.concatenate([self.V[l], v], axis=0)
            o = np.zeros((T, m.H, m.Dh), dtype=m.dtype)
            for t in range(T):
                n_keys = self.n + t + 1
                for hd in range(m.H):
                    o[t, hd] = softmax_attend(q[t, hd], self.K[l][:n_keys, hd], self.V[l][:n_keys, hd])
            h = h + o.reshape(T, m.d) @ m.w[f"l{l}.wo"].T
            h = m._ffn(l, h)
        self.n += T
        return h[-1], m.logits_of(h[-1])


# ----------------------------------------------------------------------------- generation

def generate(model: Decoder, prompt, cap: int, eos_at: int | None = None,
             keep_logits: bool = False, keep_hidden: bool = False,
             temperature: float = 0.0, seed: int = 0, row_key: int = 0) -> dict:
    """Generation of one row, at most `cap` new tokens (the first one, produced by the prompt's
    forward pass, counts).  Greedy by default; with temperature > 0 the t-th token is the draw
    (seed, row_key, t) from softmax(logits / temperature) as defined in oracle/sampler.py
    (Sec. 4.2: the paper generates at temperature 0.5).

    Termination rules (they make lengths controllable with random weights):
      * eos_at is None: natural EOS -- the row ends when argmax picks eos_id.
      * eos_at = t >= 1: the EOS logit is left out of every argmax and the t-th generated
        token is overwritten with EOS.  The response length therefore counts its EOS.
    Returns tokens (list, includes the EOS if reached), finished (EOS emitted),
    and optionally the per-step logits / final hidden states that produced each token.
    The t-th generated token (t = 1..) comes from the forward pass at position len(prompt)+t-2.
    """
    kv = KVDecoder(model)
    out, logs, hids = [], [], []
    hidden, logits = kv.feed(prompt)
    finished = False
    for t in range(1, cap + 1):
        if keep_logits:
            logs.append(logits)
        if keep_hidden:
            hids.append(hidden)
        if temperature > 0:
            tok = sample_token(logits, temperature, seed, row_key, t, model.eos_id, suppress_eos=eos_at is not None)
        else:
            tok = select_token(logits, model.eos_id, suppress_eos=eos_at is not None)
        if eos_at is not None and t == eos_at:
            tok = model.eos_id
        out.append(tok)
        if tok == model.eos_id:
            finished = True
            break
        if t < cap:
            hidden, logits = kv.feed(tok)
    return {"tokens": out, "finished": finished, "logits": logs, "hidden": hids}


def run_micro_batch(model: Decoder, prompts: list, cap: int, eos_at: list | None) -> dict:
    """One micro-batch: every row generates until its EOS or the cap; the batch lasts
    until its slowest row stops (Sec. 4.1: a batch waits for its longest member; FCR
    bounds the wait by the cap).  Rows are independent, so this is a loop over rows."""
    rows = [generate(model, p, cap, None if eos_at is None else int(eos_at[i]))
            for i, p in enumerate(prompts)]
    steps = max(len(r["tokens"]) for r in rows)
    return {"rows": rows, "steps": steps}
