"""Seeded synthetic inputs: model weights, request groups, permutations.

This module only draws numbers.  It holds none of the decoder's or the
scheduler's arithmetic, so both the CUDA path and the CPU oracle may be fed from
it without sharing any of the method between them.  It imports nothing else
from this package and needs only numpy.

Conventions
-----------
* Weights are fp32 N(0, sigma) draws rounded to the nearest bf16 value (ties to
  even).  They are returned as float32 arrays whose values are exactly
  representable in bf16, so that a consumer that stores bf16 and a consumer that
  computes in fp32/fp64 multiply identical numbers.  `to_bf16_bits` gives the
  16-bit patterns for upload.
* Norm gains are exactly 1.0.
* Response lengths count the end-of-sequence token: a target length of 1 means
  the very first generated token is EOS.
* Predicted lengths are drawn once here (true length plus Gaussian noise, rounded
  half-to-even, clamped to [1, max_new]) and stored, so every consumer reads the
  same integers.
"""
from __future__ import annotations

import dataclasses
import numpy as np


@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    eos_id: int = 2
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers)


TINY = ModelShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=1024)
LLAMA_7B = ModelShape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=32000)
LLAMA_13B = ModelShape(n_layers=40, d_model=5120, n_heads=40, head_dim=128, d_ffn=13824, vocab=32000)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 value (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _normal_bf16(rng: np.random.Generator, shape, sigma: float) -> np.ndarray:
    w = rng.standard_normal(size=shape, dtype=np.float32)
    w *= np.float32(sigma)
    return round_to_bf16(w)


def make_weights(shape: ModelShape, seed: int = 1234, sigma: float = 0.02) -> dict:
    """Random decoder weights.  All projection matrices are [out_features, in_features].

    Keys: "embed" [V,d], "lm_head" [V,d], "final_norm" [d], and per layer l:
    "l{l}.attn_norm" [d], "l{l}.wq|wk|wv|wo" [d,d], "l{l}.ffn_norm" [d],
    "l{l}.w_gate|w_up" [F,d], "l{l}.w_down" [d,F].
    """
    rng = np.random.Generator(np.random.Philox(seed))
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    assert shape.n_heads * shape.head_dim == d
    w = {"embed": _normal_bf16(rng, (V, d), sigma)}
    for l in range(shape.n_layers):
        p = f"l{l}."
        w[p + "attn_norm"] = np.ones(d, dtype=np.float32)
        w[p + "wq"] = _normal_bf16(rng, (d, d), sigma)
        w[p + "wk"] = _normal_bf16(rng, (d, d), sigma)
        w[p + "wv"] = _normal_bf16(rng, (d, d), sigma)
        w[p + "wo"] = _normal_bf16(rng, (d, d), sigma)
        w[p + "ffn_norm"] = np.ones(d, dtype=np.float32)
        w[p + "w_gate"] = _normal_bf16(rng, (F, d), sigma)
        w[p + "w_up"] = _normal_bf16(rng, (F, d), sigma)
        w[p + "w_down"] = _normal_bf16(rng, (d, F), sigma)
    w["final_norm"] = np.ones(d, dtype=np.float32)
    w["lm_head"] = _normal_bf16(rng, (V, d), sigma)
    return w


@dataclasses.dataclass
class Group:
    """One group of queries (the unit the scheduler works on)."""
    prompt_tokens: np.ndarray   # int32 [sum prompt_len], packed
    prompt_off: np.ndarray      # int64 [n+1]
    prompt_len: np.ndarray      # int32 [n]
    true_len: np.ndarray        # int32 [n], 1..max_new, counts EOS
    pred_len: np.ndarray        # int32 [n], 1..max_new
    max_new: int

    @property
    def n(self) -> int:
        return int(self.prompt_len.shape[0])

    def prompt(self, i: int) -> np.ndarray:
        return self.prompt_tokens[self.prompt_off[i]:self.prompt_off[i + 1]]


def make_group(n: int, *, vocab: int, eos_id: int, prompt_lo: int, prompt_hi: int,
               resp: str, max_new: int, noise_sigma: float, seed: int,
               resp_median: float = 120.0, resp_sigma: float = 0.7) -> Group:
    """Draw a group of n queries.

    prompt lengths ~ U{prompt_lo..prompt_hi}; prompt ids uniform over the vocabulary
    without eos_id; response lengths either "uniform" over {1..max_new} or
    "lognormal" (median resp_median, log-std resp_sigma, rounded, clipped to
    [1, max_new]); predicted = true + noise_sigma * z, rounded half-to-even, clamped.
    """
    rng = np.random.Generator(np.random.Philox(seed))
    prompt_len = rng.integers(prompt_lo, prompt_hi + 1, size=n).astype(np.int32)
    off = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(prompt_len, out=off[1:])
    ids = rng.integers(0, vocab - 1, size=int(off[-1])).astype(np.int32)
    ids[ids >= eos_id] += 1            # skip eos_id
    if resp == "uniform":
        true_len = rng.integers(1, max_new + 1, size=n)
    elif resp == "lognormal":
        x = np.exp(np.log(resp_median) + resp_sigma * rng.standard_normal(size=n))
        true_len = np.rint(x)
    else:
        raise ValueError(resp)
    true_len = np.clip(true_len, 1, max_new).astype(np.int32)
    z = rng.standard_normal(size=n)
    pred = np.rint(true_len.astype(np.float64) + noise_sigma * z)
    pred_len = np.clip(pred, 1, max_new).astype(np.int32)
    return Group(ids, off, prompt_len, true_len, pred_len, max_new)


def make_permutation(n: int, seed: int) -> np.ndarray:
    """Seeded random order of the group for the vanilla (unscheduled) arm."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.permutation(n).astype(np.int32)


# The workloads of the evaluation, by name.  Prompt/response shapes stand in for the
# instruction-following sets the paper measured on (short prompts, right-skewed
# responses truncated at 512, a longer-tailed set truncated at 2048).
def group_tiny(seed: int = 0) -> Group:
    return make_group(32, vocab=TINY.vocab, eos_id=TINY.eos_id, prompt_lo=8, prompt_hi=32,
                      resp="uniform", max_new=64, noise_sigma=8.0, seed=seed)


def group_7b_batch16(seed: int = 0) -> Group:
    return make_group(16, vocab=LLAMA_7B.vocab, eos_id=LLAMA_7B.eos_id, prompt_lo=64, prompt_hi=256,
                      resp="lognormal", max_new=512, noise_sigma=40.0, seed=seed)


def group_7b_1024(seed: int = 0) -> Group:
    return make_group(1024, vocab=LLAMA_7B.vocab, eos_id=LLAMA_7B.eos_id, prompt_lo=64, prompt_hi=256,
                      resp="lognormal", max_new=512, noise_sigma=40.0, seed=seed)


def group_13b_512(seed: int = 0) -> Group:
    return make_group(512, vocab=LLAMA_13B.vocab, eos_id=LLAMA_13B.eos_id, prompt_lo=64, prompt_hi=512,
                      resp="lognormal", max_new=2048, noise_sigma=40.0, seed=seed,
                      resp_median=200.0)
