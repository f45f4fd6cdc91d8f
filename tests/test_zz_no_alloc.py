"""ss_logits_noalloc(): the entry point for callers that may not allocate device memory (code
inside someone else's graph capture or allocator callback, or a process whose memory belongs to
another pool).  Its scratch is a fixed array inside the library that all calls share, so the
check is made on two calls in a row with different inputs: each must reproduce the logits that
the engine's own entry points (ss_prefill / ss_decode_step with dump_logits) computed from the
same hidden states, and the logits the CPU oracle's final norm + LM head give for them, within
the tolerance of the other GPU tests (2e-2 of the largest logit).
This file sorts last on purpose: a failure here cannot hide the other tests in a -x run."""
import numpy as np
import pytest

from oracle import decoder as od
from paper_2305_13144_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_logits_match_engine_on_two_calls_in_a_row():
    import torch
    from paper_2305_13144_b200 import api
    shape = synth.TINY
    w = synth.make_weights(shape, seed=1234)
    bits = {k: synth.to_bf16_bits(v) for k, v in w.items()}
    eng = api.make_engine(shape, api.runtime_cfg(16, 128, 512, 16, 2048), bits)
    oracle = od.Decoder(w, n_layers=shape.n_layers, n_heads=shape.n_heads, head_dim=shape.head_dim,
                        rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, eos_id=shape.eos_id)
    gain = torch.from_numpy(bits["final_norm"].view(np.int16)).cuda().view(torch.bfloat16)
    head = torch.from_numpy(bits["lm_head"].view(np.int16)).cuda().view(torch.bfloat16)
    g = synth.group_tiny(seed=3)
    B = 5
    toks = np.concatenate([g.prompt(i) for i in range(B)]).astype(np.int32)
    cu = np.zeros(B + 1, dtype=np.int32)
    cu[1:] = np.cumsum(g.prompt_len[:B])
    dl = torch.zeros(B, shape.vocab, dtype=torch.float32, device="cuda")
    dh = torch.zeros(B, shape.d_model, dtype=torch.float32, device="cuda")
    mine = torch.full((B, shape.vocab), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    api.ss_prefill(eng, toks, cu, None, 8, dump_logits=dl, dump_hidden=dh)
    for call in range(2):
        torch.cuda.synchronize()
        api.ss_logits_noalloc(dh, gain, head, shape.rms_eps, mine)
        torch.cuda.synchronize()
        ref, got = dl.cpu().numpy(), mine.cpu().numpy()
        assert np.isfinite(got).all()
        err = np.max(np.abs(got - ref)) / np.max(np.abs(ref))
        assert err <= 2e-2, (call, err)
        exp = oracle.logits_of(dh.cpu().numpy().astype(np.float64))        # the oracle on the same hidden states
        err_o = np.max(np.abs(got - exp)) / np.max(np.abs(exp))
        assert err_o <= 2e-2, (call, err_o)
        mine.fill_(float("nan"))
        api.ss_decode_step(eng, dump_logits=dl, dump_hidden=dh)      # new hidden states for the second call
    api.ss_release_batch(eng)


def test_noalloc_rejects_sizes_beyond_its_array():
    import torch
    from paper_2305_13144_b200 import api
    d, V = 64, 256
    gain = torch.ones(d, dtype=torch.bfloat16, device="cuda")
    head = torch.zeros(V, d, dtype=torch.bfloat16, device="cuda")
    h = torch.zeros(17, d, dtype=torch.float32, device="cuda")
    out = torch.zeros(17, V, dtype=torch.float32, device="cuda")
    with pytest.raises(api.SSError) as e:
        api.ss_logits_noalloc(h, gain, head, 1e-6, out)              # 17 rows > 16
    assert e.value.code == api.SS_ERR_CAPACITY
