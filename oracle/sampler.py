"""CPU oracle for sampled decoding at a temperature.  TEST INFRASTRUCTURE ONLY.

The paper generates at temperature 0.5 (Sec. 4.2, "Experimental Setting"; Sec. 3.2 discusses the spread of
lengths between generations that follows from sampling).  A sampled token is a draw from softmax(logits / T).
The draw is written here as the Gumbel-max form of that same distribution,

    token = argmax_v ( logit_v / T + g_v ),   g_v = -log(-log(u_v)),   u_v uniform on (0, 1),

because then every u_v can come from a counter-based generator keyed by what the draw belongs to --
(seed, query, index of the generated token, vocabulary id) -- and a parallel implementation that evaluates the
vocabulary in any order, or regenerates a row from its prompt, reproduces the same token.  Ties go to the lowest
id, a suppressed EOS is left out, and T = 0 means greedy.

The generator is Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
SC'11), written from its published definition: ten rounds of
    (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0))
with M0 = 0xD2511F53, M1 = 0xCD9E8D57 and the key advanced by (0x9E3779B9, 0xBB67AE85) between rounds.
Counter = (vocabulary id, generated-token index (1-based), query key, 0); key = (seed low word, seed high word).
u = ((first output word >> 9) + 0.5) / 2^23, which is exact in single precision and never 0 or 1.

Pins (tests/test_oracle_sampler.py): the generator's published known-answer vectors; T = 0 and T -> 0 give the
greedy choice; over 1e5 counters the frequency of each token matches softmax(logits / T) within three standard
errors (two logits, and five logits by chi-square); the same counter gives the same token; EOS suppression.
This file imports nothing from the CUDA package.
"""
from __future__ import annotations

import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_W0, _W1 = np.uint64(0x9E3779B9), np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32 with ten rounds on arrays (or scalars) of 32-bit words held in uint64.  Returns four words."""
    c0, c1, c2, c3, k0, k1 = (np.asarray(a, dtype=np.uint64) & _MASK for a in (c0, c1, c2, c3, k0, k1))
    for r in range(10):
        if r > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0                      # 32 x 32 -> 64 bits, exact in uint64
        p1 = _M1 * c2
        c0, c1, c2, c3 = ((p1 >> _S32) ^ c1 ^ k0) & _MASK, p1 & _MASK, ((p0 >> _S32) ^ c3 ^ k1) & _MASK, p0 & _MASK
    return c0, c1, c2, c3


def uniform_open(word):
    """A 32-bit word -> a uniform number in (0, 1): ((word >> 9) + 0.5) / 2^23 (24 significant bits)."""
    return ((np.asarray(word, dtype=np.uint64) >> np.uint64(9)).astype(np.float64) + 0.5) / float(1 << 23)


def gumbel_noise(seed: int, row_key: int, step: int, vocab: int) -> np.ndarray:
    """g_v for v = 0..vocab-1 of the draw (seed, row_key, step)."""
    v = np.arange(vocab, dtype=np.uint64)
    w0, _, _, _ = philox4x32_10(v, np.uint64(step), np.uint64(row_key), np.uint64(0),
                                np.uint64(seed & 0xFFFFFFFF), np.uint64((seed >> 32) & 0xFFFFFFFF))
    return -np.log(-np.log(uniform_open(w0)))


def perturbed(logits: np.ndarray, temperature: float, seed: int, row_key: int, step: int) -> np.ndarray:
    """logits / T + g: the quantity whose arg-max is the sampled token (T > 0)."""
    return np.asarray(logits, dtype=np.float64) / float(temperature) + gumbel_noise(seed, row_key, step, len(logits))


def sample_token(logits: np.ndarray, temperature: float, seed: int, row_key: int, step: int, eos_id: int,
                 suppress_eos: bool) -> int:
    """One draw from softmax(logits / T) (lowest id on ties; EOS left out when suppressed); greedy at T = 0."""
    if np.isnan(logits).any():
        raise FloatingPointError("NaN logit")
    z = np.asarray(logits, dtype=np.float64).copy() if temperature == 0 else perturbed(logits, temperature, seed, row_key, step)
    if suppress_eos:
        z[eos_id] = -np.inf
    return int(np.argmax(z))
