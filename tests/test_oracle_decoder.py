"""Pins for the decoder oracle: closed forms, hand-worked fixtures, brute force on tiny
inputs and the three-route invariants.  No GPU, no CUDA code."""
import json
import math
import os

import numpy as np
import pytest

from oracle import decoder as od
from paper_2305_13144_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


# ------------------------------------------------------------------ attention

def test_attention_ln_weights_fixture():
    g = _gold("attention_ln_weights.json")
    q = np.array(g["q"])
    K = np.array([[math.log(j), 7.0, -3.0, 0.5] for j in g["k_first_coord_times_ln"]])
    V = np.array(g["v"])
    out = od.softmax_attend(q, K, V)
    np.testing.assert_allclose(out, g["out"], rtol=0, atol=1e-12)


def test_attention_one_key_returns_value():
    rng = np.random.default_rng(0)
    q, k, v = rng.normal(size=8), rng.normal(size=(1, 8)), rng.normal(size=(1, 8))
    np.testing.assert_array_equal(od.softmax_attend(q, k, v), v[0])


def test_attention_identical_keys_give_mean_value():
    rng = np.random.default_rng(1)
    q, k = rng.normal(size=8), rng.normal(size=8)
    V = rng.normal(size=(5, 8))
    out = od.softmax_attend(q, np.tile(k, (5, 1)), V)
    np.testing.assert_allclose(out, V.mean(axis=0), atol=1e-14)


def test_attention_masked_key_changes_nothing_and_shift_invariance():
    rng = np.random.default_rng(2)
    q, K, V = rng.normal(size=16), rng.normal(size=(6, 16)), rng.normal(size=(6, 16))
    base = od.softmax_attend(q, K, V)
    K2 = np.vstack([K, rng.normal(size=(1, 16)) * 50])
    V2 = np.vstack([V, rng.normal(size=(1, 16)) * 50])
    bias = np.array([0.0] * 6 + [-np.inf])
    np.testing.assert_allclose(od.softmax_attend(q, K2, V2, bias), base, atol=1e-14)
    # a constant added to every score cancels
    np.testing.assert_allclose(od.softmax_attend(q, K, V, np.full(6, 123.0)), base, atol=1e-12)


def test_attention_brute_force_scalar_loops():
    rng = np.random.default_rng(3)
    for n, dh in [(1, 2), (3, 4), (17, 8)]:
        q, K, V = rng.normal(size=dh), rng.normal(size=(n, dh)), rng.normal(size=(n, dh))
        scores = [sum(q[i] * K[j][i] for i in range(dh)) / math.sqrt(dh) for j in range(n)]
        z = sum(math.exp(s) for s in scores)
        ref = [sum(math.exp(scores[j]) / z * V[j][i] for j in range(n)) for i in range(dh)]
        np.testing.assert_allclose(od.softmax_attend(q, K, V), ref, rtol=1e-12, atol=1e-13)


def test_attention_large_scores_do_not_overflow():
    q = np.array([1000.0, 0.0])
    K = np.array([[1.0, 0.0], [2.0, 0.0]])
    V = np.array([[1.0, 0.0], [0.0, 1.0]])
    out = od.softmax_attend(q, K, V)
    assert np.isfinite(out).all() and out[1] > 0.999999


# ------------------------------------------------------------------ RoPE

def test_rope_fixture_dh4():
    g = _gold("rope_dh4.json")
    for c in g["cases"]:
        x = np.array(c["x"])
        a0, a1 = c["angles"]
        exp = [x[0] * math.cos(a0) - x[2] * math.sin(a0),
               x[1] * math.cos(a1) - x[3] * math.sin(a1),
               x[2] * math.cos(a0) + x[0] * math.sin(a0),
               x[3] * math.cos(a1) + x[1] * math.sin(a1)]
        got = od.rope(x, np.array(c["pos"]), g["theta"])
        np.testing.assert_allclose(got, exp, atol=1e-13)


def test_rope_dh2_is_plane_rotation():
    got = od.rope(np.array([1.0, 0.0]), np.array(2), 10000.0)
    np.testing.assert_allclose(got, [math.cos(2.0), math.sin(2.0)], atol=1e-15)


def test_rope_identity_norm_and_relative_property():
    rng = np.random.default_rng(4)
    q, k = rng.normal(size=64), rng.normal(size=64)
    np.testing.assert_array_equal(od.rope(q, np.array(0), 10000.0), q)
    for p in (1, 17, 700):
        assert abs(np.linalg.norm(od.rope(q, np.array(p), 10000.0)) - np.linalg.norm(q)) < 1e-12
    d1 = od.rope(q, np.array(9), 1e4) @ od.rope(k, np.array(4), 1e4)
    d2 = od.rope(q, np.array(309), 1e4) @ od.rope(k, np.array(304), 1e4)
    assert abs(d1 - d2) < 1e-10
    d3 = od.rope(q, np.array(10), 1e4) @ od.rope(k, np.array(4), 1e4)
    assert abs(d1 - d3) > 1e-6          # and it does depend on the distance


def test_rope_broadcast_over_heads_and_tokens():
    rng = np.random.default_rng(5)
    x = rng.normal(size=(3, 2, 8))
    pos = np.array([0, 5, 9])
    got = od.rope(x, pos[:, None], 1e4)
    for t in range(3):
        for h in range(2):
            np.testing.assert_allclose(got[t, h], od.rope(x[t, h], np.array(pos[t]), 1e4), atol=1e-15)


# ------------------------------------------------------------------ RMSNorm, SiLU, argmax

def test_rmsnorm_properties():
    rng = np.random.default_rng(6)
    x = rng.normal(size=(4, 32))
    g = np.ones(32)
    y = od.rmsnorm(x, g, 0.0)
    np.testing.assert_allclose(np.sqrt((y * y).mean(axis=-1)), 1.0, atol=1e-14)
    np.testing.assert_allclose(od.rmsnorm(3.7 * x, g, 0.0), y, atol=1e-14)
    c = od.rmsnorm(np.full(8, -2.5), np.arange(1.0, 9.0), 0.0)
    np.testing.assert_allclose(c, -np.arange(1.0, 9.0), atol=1e-14)
    # eps sits inside the square root, added to the mean square
    np.testing.assert_allclose(od.rmsnorm(np.array([3.0, 4.0]), np.ones(2), 3.5),
                               np.array([3.0, 4.0]) / 4.0, atol=1e-15)


def test_silu_identities():
    assert od.silu(np.array(0.0)) == 0.0
    x = np.linspace(-6, 6, 25)
    np.testing.assert_allclose(od.silu(x) - od.silu(-x), x, atol=1e-14)
    assert abs(od.silu(np.array(40.0)) - 40.0) < 1e-12
    assert abs(od.silu(np.array(1.0)) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15


def test_select_token_ties_and_eos():
    assert od.select_token(np.zeros(7), eos_id=2, suppress_eos=False) == 0
    l = np.zeros(7); l[2] = 5.0; l[5] = 5.0
    assert od.select_token(l, eos_id=2, suppress_eos=False) == 2
    assert od.select_token(l, eos_id=2, suppress_eos=True) == 5
    l0 = np.zeros(4)
    assert od.select_token(l0, eos_id=0, suppress_eos=True) == 1
    with pytest.raises(FloatingPointError):
        od.select_token(np.array([0.0, np.nan]), 0, False)


# ------------------------------------------------------------------ whole model

def _tiny_shape():
    return synth.ModelShape(n_layers=2, d_model=8, n_heads=2, head_dim=4, d_ffn=6, vocab=11, eos_id=2)


def _model(shape, w, dtype=np.float64):
    return od.Decoder(w, n_layers=shape.n_layers, n_heads=shape.n_heads, head_dim=shape.head_dim,
                      rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, eos_id=shape.eos_id, dtype=dtype)


def _scalar_reference(shape, w, tokens):
    """The same decoder in scalar Python loops, written independently of numpy's matmul
    orientation; feasible only at toy sizes."""
    d, H, Dh, F = shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn
    eps, theta = shape.rms_eps, shape.rope_theta
    T = len(tokens)

    def norm(x, g):
        r = math.sqrt(sum(v * v for v in x) / len(x) + eps)
        return [x[i] / r * g[i] for i in range(len(x))]

    def matvec(W, x):  # W [out][in]
        return [sum(W[o][i] * x[i] for i in range(len(x))) for o in range(len(W))]

    def rot(x, p):     # one head
        out = list(x)
        for i in range(Dh // 2):
            a = p * theta ** (-2.0 * i / Dh)
            out[i] = x[i] * math.cos(a) - x[i + Dh // 2] * math.sin(a)
            out[i + Dh // 2] = x[i + Dh // 2] * math.cos(a) + x[i] * math.sin(a)
        return out

    h = [[float(v) for v in w["embed"][t]] for t in tokens]
    for l in range(shape.n_layers):
        qs, ks, vs = [], [], []
        for p in range(T):
            u = norm(h[p], w[f"l{l}.attn_norm"])
            q, k, v = matvec(w[f"l{l}.wq"], u), matvec(w[f"l{l}.wk"], u), matvec(w[f"l{l}.wv"], u)
            qs.append([rot(q[a * Dh:(a + 1) * Dh], p) for a in range(H)])
            ks.append([rot(k[a * Dh:(a + 1) * Dh], p) for a in range(H)])
            vs.append([v[a * Dh:(a + 1) * Dh] for a in range(H)])
        for p in range(T):
            o = []
            for a in range(H):
                sc = [sum(qs[p][a][i] * ks[j][a][i] for i in range(Dh)) / math.sqrt(Dh) for j in range(p + 1)]
                z = sum(math.exp(s) for s in sc)
                o += [sum(math.exp(sc[j]) / z * vs[j][a][i] for j in range(p + 1)) for i in range(Dh)]
            att = matvec(w[f"l{l}.wo"], o)
            h[p] = [h[p][i] + att[i] for i in range(d)]
        for p in range(T):
            u2 = norm(h[p], w[f"l{l}.ffn_norm"])
            g, up = matvec(w[f"l{l}.w_gate"], u2), matvec(w[f"l{l}.w_up"], u2)
            a = [g[i] / (1.0 + math.exp(-g[i])) * up[i] for i in range(F)]
            dn = matvec(w[f"l{l}.w_down"], a)
            h[p] = [h[p][i] + dn[i] for i in range(d)]
    logits = [matvec(w["lm_head"], norm(h[p], w["final_norm"])) for p in range(T)]
    return h, logits


def test_full_forward_against_scalar_loops():
    shape = _tiny_shape()
    w = synth.make_weights(shape, seed=7, sigma=0.5)      # large sigma: every term matters
    for l in range(shape.n_layers):                      # non-trivial gains, too
        w[f"l{l}.attn_norm"] = np.linspace(0.5, 1.5, shape.d_model).astype(np.float32)
        w[f"l{l}.ffn_norm"] = np.linspace(1.5, 0.5, shape.d_model).astype(np.float32)
    w["final_norm"] = np.linspace(0.8, 1.2, shape.d_model).astype(np.float32)
    tokens = [3, 9, 0, 5, 5]
    m = _model(shape, w)
    h, logits = m.forward_full(tokens)
    h_ref, logits_ref = _scalar_reference(shape, {k: v.astype(np.float64) for k, v in w.items()}, tokens)
    np.testing.assert_allclose(h, h_ref, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(logits, logits_ref, rtol=1e-10, atol=1e-11)


def test_zero_output_projections_closed_form():
    shape = synth.TINY
    w = synth.make_weights(shape, seed=11)
    for l in range(shape.n_layers):
        w[f"l{l}.wo"][:] = 0
        w[f"l{l}.w_down"][:] = 0
    m = _model(shape, w)
    tokens = [5, 77, 1000, 3]
    h, logits = m.forward_full(tokens)
    E = w["embed"].astype(np.float64)[tokens]
    np.testing.assert_array_equal(h, E)
    exp = (E / np.sqrt((E * E).mean(-1, keepdims=True) + shape.rms_eps)) @ w["lm_head"].astype(np.float64).T
    np.testing.assert_allclose(logits, exp, atol=1e-13)


def test_zero_value_projection_kills_attention_only():
    shape = _tiny_shape()
    w = synth.make_weights(shape, seed=12, sigma=0.5)
    for l in range(shape.n_layers):
        w[f"l{l}.wv"][:] = 0
    m = _model(shape, w)
    # with Wv = 0 tokens cannot see each other: each position equals its solo run
    h, _ = m.forward_full([4, 8, 1])
    for p, t in enumerate([4, 8, 1]):
        h1, _ = m.forward_full([t])
        np.testing.assert_allclose(h[p], h1[0], atol=1e-13)


def test_zero_layers_is_embedding_lookup():
    shape = _tiny_shape().with_layers(0)
    w = synth.make_weights(shape, seed=13)
    m = _model(shape, w)
    h, _ = m.forward_full([1, 2, 3])
    np.testing.assert_array_equal(h, w["embed"].astype(np.float64)[[1, 2, 3]])


def test_kv_cache_equals_recomputation_tiny_config():
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    m = _model(shape, w)
    g = synth.group_tiny(seed=0)
    prompt = g.prompt(0).tolist()
    r = od.generate(m, prompt, cap=12, eos_at=12, keep_logits=True, keep_hidden=True)
    seq = prompt + r["tokens"][:-1]
    h_full, logit_full = m.forward_full(seq)
    for t in range(len(r["tokens"])):
        p = len(prompt) + t - 1
        np.testing.assert_allclose(r["hidden"][t], h_full[p], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(r["logits"][t], logit_full[p], rtol=1e-9, atol=1e-12)
    # and the greedy tokens follow from the recomputed logits
    for t, tok in enumerate(r["tokens"][:-1]):
        assert tok == od.select_token(logit_full[len(prompt) + t - 1], shape.eos_id, True)
    assert r["tokens"][-1] == shape.eos_id and r["finished"]


def test_batch_padding_leaves_rows_unchanged():
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    m = _model(shape, w)
    g = synth.group_tiny(seed=1)
    seqs = [g.prompt(i).tolist()[:4 + 2 * i] for i in range(4)]       # unequal lengths 4..10
    hb, lb = m.forward_padded(seqs)
    for i, s in enumerate(seqs):
        h1, l1 = m.forward_full(s)
        np.testing.assert_allclose(hb[i], h1[-1], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(lb[i], l1[-1], rtol=1e-9, atol=1e-12)


def test_generate_termination_rules():
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    m = _model(shape, w)
    p = synth.group_tiny(seed=0).prompt(3).tolist()
    r1 = od.generate(m, p, cap=5, eos_at=1)
    assert r1["tokens"] == [shape.eos_id] and r1["finished"]
    r3 = od.generate(m, p, cap=5, eos_at=3)
    assert len(r3["tokens"]) == 3 and r3["tokens"][-1] == shape.eos_id and shape.eos_id not in r3["tokens"][:-1]
    r_cut = od.generate(m, p, cap=2, eos_at=3)
    assert len(r_cut["tokens"]) == 2 and not r_cut["finished"]
    assert r_cut["tokens"] == r3["tokens"][:2]           # the cap only truncates
    mb = od.run_micro_batch(m, [p, p], cap=4, eos_at=[2, 9])
    assert mb["steps"] == 4 and mb["rows"][0]["finished"] and not mb["rows"][1]["finished"]


def test_fp32_route_agrees_with_fp64():
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    tokens = synth.group_tiny(seed=0).prompt(1).tolist()
    _, l64 = _model(shape, w).forward_full(tokens)
    _, l32 = _model(shape, w, np.float32).forward_full(tokens)
    assert l32.dtype == np.float32
    assert np.max(np.abs(l64 - l32)) < 1e-4 * np.max(np.abs(l64))


def test_weight_generator_values_are_bf16():
    w = synth.make_weights(_tiny_shape(), seed=3)
    for k, v in w.items():
        assert v.dtype == np.float32
        assert (v.view(np.uint32) & 0xFFFF == 0).all(), k
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9], dtype=np.float32)
    # ties to even: 1+2^-8 is halfway between 1 and 1+2^-7 -> 1; 1+3*2^-8 -> 1+2^-6
    np.testing.assert_array_equal(synth.round_to_bf16(x), np.array([1.0, 1.0 + 2 ** -6, 1.0], dtype=np.float32))
