"""GPU parity at the benchmark's model shapes (cut to a few layers so that the numpy oracle finishes in
minutes): the 7B shape of configurations 2-4 and the 13B shape of configuration 5, teacher-forced on the
oracle's tokens, through the C ABI.  The oracle runs in float32 here (its float64 route is compared with it
in tests/test_oracle_decoder.py); its rounding is four orders below the tolerances, which at these shapes are
2e-2 * sqrt(layers / 2) for logits and hidden state (see parity_util.large_shape_tol and tests/test_bf16_floor.py).

What these cases reach that the small configuration does not: 128-wide heads, 32 / 40 heads, the tile and
split tables of d = 4096 / 5120 and FFN 11008 / 13824 (129 / 162 tiles of 256 rows split over the SMs along
K), a 32000-row vocabulary, contexts that cross key/value pages during decoding, rows that finish while
their neighbours continue.
"""
import numpy as np
import pytest

from paper_2305_13144_b200 import synth
from parity_util import large_shape_tol, teacher_forced

pytestmark = pytest.mark.gpu


def test_7b_shape_eight_layers_forty_steps_pages_and_finishing_rows():
    """Batch 16 with the benchmark's prompts (U[64,256]); the oracle follows the six rows with the shortest
    prompts for 41 generated tokens.  Every row's context crosses at least one 32-token page boundary on the
    way; two followed rows finish early (after 5 and 20 tokens) and two unfollowed ones (after 9 and 30) while
    the rest keep decoding, so the active mask is exercised at head size 128 (App. D: the per-token path)."""
    shape = synth.LLAMA_7B.with_layers(8)
    w = synth.make_weights(shape, seed=7)
    g = synth.group_7b_batch16(seed=0)
    B, cap = g.n, 41
    by_len = np.argsort(g.prompt_len, kind="stable").tolist()
    follow = by_len[:6]
    targets = np.full(B, 100, dtype=np.int32)              # beyond the cap: cut after 41 tokens
    targets[follow[1]], targets[follow[4]] = 5, 20
    targets[by_len[8]], targets[by_len[12]] = 9, 30
    prompts = [g.prompt(i).tolist() for i in range(B)]
    el, eh, steps = teacher_forced(shape, w, prompts, targets, cap, follow=follow, dtype=np.float32,
                                   max_batch=16, max_ctx=768, max_prefill=4096, max_new=64, kv_tokens=16 * 768)
    assert steps == cap
    tol = large_shape_tol(8)                               # 4e-2: twice the bf16 storage floor at eight layers
    assert el <= tol and eh <= tol, (el, eh)


def test_13b_shape_two_layers_batch16():
    """d 5120, 40 heads x 128, FFN 13824: 16 rows with prompts U[64,512] as in configuration 5; the oracle
    follows the four rows with the shortest prompts through the prompt pass and seven decode steps; one of
    them ends after three tokens."""
    shape = synth.LLAMA_13B.with_layers(2)
    w = synth.make_weights(shape, seed=13)
    g = synth.group_13b_512(seed=0)
    B, cap = 16, 8
    idx = list(range(B))
    follow = np.argsort(g.prompt_len[:B], kind="stable")[:4].tolist()
    targets = np.full(B, 50, dtype=np.int32)
    targets[follow[2]] = 3
    targets[5 if 5 not in follow else 6] = 2
    prompts = [g.prompt(i).tolist() for i in idx]
    el, eh, steps = teacher_forced(shape, w, prompts, targets, cap, follow=follow, dtype=np.float32,
                                   max_batch=16, max_ctx=640, max_prefill=8192, max_new=16, kv_tokens=16 * 640)
    assert steps == cap
    assert el <= large_shape_tol(2) and eh <= large_shape_tol(2), (el, eh)


@pytest.mark.parametrize("B", [48, 80])
def test_13b_shape_two_layers_attention_in_several_passes(B):
    """40 heads x 48 or 80 rows are 13 or 22 (row, head) pairs per CTA of a 148-SM part: more than the eight of one
    pass, fewer than the 24 from which every warp takes whole pairs.  48 rows run in the kernel of the batches up
    to 64 rows, 80 rows in the one for wide batches; prompts of 20 to 90 tokens, so rows differ in pages; two of
    the followed rows end early."""
    shape = synth.LLAMA_13B.with_layers(2)
    w = synth.make_weights(shape, seed=13)
    rng = np.random.default_rng(1000 + B)
    cap = 3
    lens = rng.integers(20, 91, size=B)
    prompts = [rng.integers(3, shape.vocab, size=int(n)).tolist() for n in lens]
    targets = rng.integers(2, 6, size=B).astype(np.int32)
    follow = [0, B // 3, B // 2, B - 1]
    targets[follow[1]], targets[follow[2]] = 1, 2
    el, eh, steps = teacher_forced(shape, w, prompts, targets, cap, follow=follow, dtype=np.float32,
                                   max_batch=128, max_ctx=128, max_prefill=8192, max_new=8, kv_tokens=128 * 128)
    assert steps == cap
    assert el <= large_shape_tol(2) and eh <= large_shape_tol(2), (el, eh)


def test_13b_shape_two_layers_wide_batch():
    """The variable-batch-size arm's launch configuration at the 13B shape: 136 rows (two 128-lane token
    tiles, the second with 8 rows), short prompts; the oracle follows six rows spread over both tiles.  A CTA's run
    has about 37 pairs here, so every warp takes whole pairs."""
    shape = synth.LLAMA_13B.with_layers(2)
    w = synth.make_weights(shape, seed=13)
    rng = np.random.default_rng(136)
    B, cap = 136, 3
    lens = rng.integers(8, 49, size=B)
    prompts = [rng.integers(3, shape.vocab, size=int(n)).tolist() for n in lens]
    targets = rng.integers(1, 5, size=B).astype(np.int32)
    follow = [0, 63, 64, 127, 128, 135]
    targets[63], targets[128] = 2, 4
    el, eh, steps = teacher_forced(shape, w, prompts, targets, cap, follow=follow, dtype=np.float32,
                                   max_batch=256, max_ctx=128, max_prefill=8192, max_new=8, kv_tokens=256 * 64)
    assert steps == cap
    assert el <= large_shape_tol(2) and eh <= large_shape_tol(2), (el, eh)


def test_many_heads_long_contexts_pages_beyond_the_first_64():
    """A one-layer decoder with 32 heads x 64 and 120 rows whose prompts all have 2050 to 2110 tokens: 26 (row,
    head) pairs per CTA, so every warp takes whole pairs, and 65 or 66 pages per row, so the scan goes through the
    page ids a warp's lanes hold (pages 0..31 and 32..63) and the ones it looks up one by one beyond them."""
    shape = synth.ModelShape(n_layers=1, d_model=2048, n_heads=32, head_dim=64, d_ffn=512, vocab=1024)
    w = synth.make_weights(shape, seed=21)
    rng = np.random.default_rng(2100)
    B, cap = 120, 3
    lens = rng.integers(2050, 2111, size=B)
    prompts = [rng.integers(3, shape.vocab, size=int(n)).tolist() for n in lens]
    targets = rng.integers(2, 6, size=B).astype(np.int32)
    follow = [0, 59, 119]
    targets[59] = 2
    el, eh, steps = teacher_forced(shape, w, prompts, targets, cap, follow=follow, dtype=np.float32,
                                   max_batch=128, max_ctx=2176, max_prefill=8192, max_new=8, kv_tokens=128 * 2176)
    assert steps == cap
    assert el <= large_shape_tol(2) and eh <= large_shape_tol(2), (el, eh)
