"""Why the tolerances at the 7B / 13B shapes are 2e-2 * sqrt(layers / 2) (and 1e-2 / 2e-2 on the small configuration).

The GPU path keeps the residual stream and every accumulation in fp32 but must store in bf16 what the tensor
cores and the cache hold: the normalised inputs of the projections, the cached keys and values, the attention
output and the SwiGLU output.  This test repeats the ORACLE's arithmetic with nothing changed but a
round-to-nearest-even to bf16 at exactly those values, on the 7B shape cut to two layers with the synthetic
N(0, 0.02) weights, and measures the relative L2 distance of the final hidden states from the unrounded run.

With these weights a projection of a unit-RMS input has RMS 0.02 * sqrt(4096) = 1.28, so after the first layer the
residual stream consists of projection outputs (RMS about 3) and no longer of the embedding (RMS 0.02): every
rounding of an operand reaches the hidden state at full relative size, attention scores of RMS 1.6 carry it through
the softmax, and the six storage points of a layer add up.  The floor measured here is about 1e-2 at two layers
(0.9e-2 to 1.2e-2 depending on the position), i.e. at the 1e-2 the small configuration meets, and it grows with the
square root of the depth.  The GPU tests at these shapes therefore allow 2e-2 * sqrt(layers / 2) for the hidden state
and for the logits (relative to the largest logit): twice the mean floor, which leaves room for the floor's own spread
over positions and for the kernels' contribution (accumulation order, fast exp, fp32 partial sums).  No GPU is involved.
"""
import numpy as np

from oracle import decoder as od
from paper_2305_13144_b200 import synth

POINTS = ("norm_attn", "q", "k", "v", "attn_out", "norm_ffn", "ffn_act")


def _forward(model, tokens, rounded=()):
    """The oracle's full-prefix route with causal attention written as one masked matrix product per head and
    an optional bf16 rounding at the named storage points."""
    def st(a, name):
        return synth.round_to_bf16(a).astype(model.dtype) if name in rounded else a
    w, T = model.w, len(tokens)
    pos = np.arange(T)
    causal = np.tril(np.ones((T, T), dtype=bool))
    h = w["embed"][np.asarray(tokens)].copy()
    for l in range(model.L):
        u = st(od.rmsnorm(h, w[f"l{l}.attn_norm"], model.eps), "norm_attn")
        q = (u @ w[f"l{l}.wq"].T).reshape(T, model.H, model.Dh)
        k = (u @ w[f"l{l}.wk"].T).reshape(T, model.H, model.Dh)
        v = (u @ w[f"l{l}.wv"].T).reshape(T, model.H, model.Dh)
        q = st(od.rope(q, pos[:, None], model.theta), "q")
        k = st(od.rope(k, pos[:, None], model.theta), "k")
        v = st(v, "v")
        o = np.empty_like(q)
        for hd in range(model.H):
            s = np.where(causal, q[:, hd] @ k[:, hd].T / np.sqrt(model.Dh), -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            o[:, hd] = (p / p.sum(axis=1, keepdims=True)) @ v[:, hd]
        h = h + st(o, "attn_out").reshape(T, model.d) @ w[f"l{l}.wo"].T
        u2 = st(od.rmsnorm(h, w[f"l{l}.ffn_norm"], model.eps), "norm_ffn")
        a = st(od.silu(u2 @ w[f"l{l}.w_gate"].T) * (u2 @ w[f"l{l}.w_up"].T), "ffn_act")
        h = h + a @ w[f"l{l}.w_down"].T
    return h


def _model(w, n_layers):
    shape = synth.LLAMA_7B
    return od.Decoder(w, n_layers=n_layers, n_heads=shape.n_heads, head_dim=shape.head_dim, rms_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, eos_id=shape.eos_id, dtype=np.float32)


def _rel(a, b):
    return np.linalg.norm(a - b, axis=1) / np.linalg.norm(b, axis=1)


def test_bf16_storage_alone_costs_one_percent_at_two_layers_and_grows_with_the_root_of_the_depth():
    shape = synth.LLAMA_7B.with_layers(4)
    w = synth.make_weights(shape, seed=7)
    tokens = np.random.default_rng(1).integers(3, shape.vocab, size=48)
    # ---- two layers (the first two of the same weights)
    model = _model(w, 2)
    exact = _forward(model, tokens)
    # the restatement above is the oracle's decoder: same hidden states as its own full-prefix route
    h_oracle, _ = model.forward_full(tokens[:12])
    assert np.max(np.abs(exact[:12] - h_oracle)) <= 1e-4 * np.max(np.abs(h_oracle))
    stored = _forward(model, tokens, rounded=POINTS)
    err = _rel(stored, exact)
    # positions 0..3 attend over one to four keys and sit lower; the rest is the floor
    floor2 = float(np.mean(err[4:]))
    assert 0.8e-2 <= floor2 <= 1.3e-2, err
    assert float(np.max(err)) > 1.0e-2, err               # some position is already above 1e-2 from storage alone
    assert float(np.max(err)) <= 2.0e-2, err              # and the 2e-2 the GPU tests allow leaves room above it
    # one storage point alone stays well below the sum: the floor comes from their number, not from one of them
    one = _forward(model, tokens, rounded=("attn_out",))
    assert float(np.mean(_rel(one, exact)[4:])) < 0.5e-2
    # ---- four layers: every layer adds its six roundings to a stream the next layer renormalises, so the
    # floor grows like the square root of the depth (measured with this same code: 0.96e-2, 1.39e-2, 1.94e-2 at
    # 2, 4, 8 layers for the hidden state; 1.93e-2 of max|logit| for the logits at 8 layers, 2.7e-2 at the worst
    # position).  The GPU tests at these shapes therefore allow 2e-2 * sqrt(layers / 2), twice the mean floor.
    model4 = _model(w, 4)
    exact4 = _forward(model4, tokens)
    stored4 = _forward(model4, tokens, rounded=POINTS)
    floor4 = float(np.mean(_rel(stored4, exact4)[4:]))
    assert 1.25 <= floor4 / floor2 <= 1.6, (floor2, floor4)
    lg_e, lg_s = model4.logits_of(exact4), model4.logits_of(stored4)
    lerr = np.max(np.abs(lg_s - lg_e), axis=1) / np.max(np.abs(lg_e), axis=1)
    assert 0.9e-2 <= float(np.mean(lerr[4:])) <= 1.9e-2, lerr      # the logits carry the same relative error
