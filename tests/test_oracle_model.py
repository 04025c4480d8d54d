"""Pins for the oracle's looped-LM forward and its depth-indexed KV (Sec. 3.1, Eq. 1; App. B).

The incremental, cached path (prefill + row-by-row advance) must equal a cache-free
full-sequence forward written here with torch float64 library routines
(scaled_dot_product_attention, silu, complex-number rotary) run with r recurrences.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as W
from oracle import numerics as nm
from oracle.loopspec import Decoder
from oracle.model import LoopedLM


def torch_full_forward(shape, w, ids, n_rec):
    """Cache-free forward of the whole sequence through n_rec recurrences; returns logits [n, V]."""
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    n = len(ids)
    d, nq, nkv = shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    x = t(w["embed"])[torch.tensor(np.asarray(ids), dtype=torch.long)]
    inv = shape.rope_theta ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    rot = torch.polar(torch.ones(n, d // 2, dtype=torch.float64),
                      torch.arange(n, dtype=torch.float64)[:, None] * inv)      # e^{i pos w}

    def rms(v, g):
        return v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * t(g)

    def rotary(v):                                   # v [n, heads, d], pairs (i, i + d/2)
        c = torch.complex(v[..., : d // 2], v[..., d // 2:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    for _ in range(n_rec):
        for l in range(shape.n_recurrent):
            g = lambda k: w[f"layers.{l}.{k}"]
            y = rms(x, g("norm1")) @ t(g("wqkv")).T
            q = rotary(y[:, : nq * d].reshape(n, nq, d)).transpose(0, 1)
            k = rotary(y[:, nq * d:(nq + nkv) * d].reshape(n, nkv, d)).transpose(0, 1)
            v = y[:, (nq + nkv) * d:].reshape(n, nkv, d).transpose(0, 1)
            k = k.repeat_interleave(nq // nkv, dim=0)
            v = v.repeat_interleave(nq // nkv, dim=0)
            a = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True)[0]
            x = x + a.transpose(0, 1).reshape(n, nq * d) @ t(g("wo")).T
            gu = rms(x, g("norm2")) @ t(g("wgateup")).T
            x = x + (F.silu(gu[:, : shape.ffn]) * gu[:, shape.ffn:]) @ t(g("wdown")).T
    head = w["embed"] if shape.tied else w["lm_head"]
    return (rms(x, w["final_norm"]) @ t(head).T).numpy()


SHAPES = {
    "mha": W.CONFIGS["tiny"].with_(vocab=64, hidden=64, n_q_heads=2, n_kv_heads=2, head_dim=32, ffn=96, R=3),
    "gqa": W.CONFIGS["tiny"].with_(vocab=64, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=80, R=3,
                                   tied=False, n_recurrent=3),
}


@pytest.mark.parametrize("name", list(SHAPES))
def test_incremental_equals_cache_free_forward(name):
    shape = SHAPES[name]
    w = W.make_weights(shape, seed=3, gain_jitter=0.1)
    model = LoopedLM(shape, w, kv_bf16=False)
    prompt = W.make_prompt(shape.vocab, 7, seed=5)
    dec = Decoder(model)
    dec.prefill(prompt, 6)
    toks, logits = dec.vanilla(5, keep_logits=True)
    ids = dec.ids
    # every decoded position's depth-R logits equal the library forward of the full prefix
    full = torch_full_forward(shape, w, ids[:-1], shape.R)
    np.testing.assert_allclose(dec.first_logits, full[len(prompt) - 1], rtol=0, atol=1e-11)
    for i, z in enumerate(logits):
        np.testing.assert_allclose(z, full[len(prompt) + i], rtol=0, atol=1e-11)
    assert [int(np.argmax(full[len(prompt) - 1 + i])) for i in range(6)] == ids[len(prompt):]


def test_early_depth_readout_is_same_C_at_depth_r():
    """p_r = C(H^r): the oracle's first-proposal logits at d1 equal the library forward with d1 recurrences."""
    shape = SHAPES["mha"]
    w = W.make_weights(shape, seed=4)
    model = LoopedLM(shape, w, kv_bf16=False)
    prompt = W.make_prompt(shape.vocab, 5, seed=6)
    for d1 in (1, 2):
        dec2 = Decoder(model)
        dec2.prefill(prompt, 4)
        dec2.active = []
        b = dec2._spawn(None, dec2.ids[-1], len(dec2.ids) - 1)
        for r in range(1, d1 + 1):
            X, own = model.advance_rows(b.H[None], [b.pos], lambda i, l: dec2._prefix_kv(b, r, l))
            b.H = X[0]
            dec2._store_committed(r, b.pos, own[0])
        full = torch_full_forward(shape, w, dec2.ids, d1)
        np.testing.assert_allclose(model.logits(b.H), full[-1], rtol=0, atol=1e-11)


def test_round_bf16_matches_torch():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000),
                        [1.00390625, 1.01171875, -1.00390625, 0.0, 65280.0]])
    ref = torch.tensor(a, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(nm.round_bf16(a), ref)
    np.testing.assert_array_equal(W.bf16_round(a.astype(np.float32)).astype(np.float64), ref)


def test_rope_is_a_rotation_and_relative():
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal((1, 1, 64)), rng.standard_normal((1, 1, 64))
    for m, n in [(3, 1), (103, 101), (5000, 4998)]:
        qm, kn = nm.rope(q, np.array([m]), 1e4), nm.rope(k, np.array([n]), 1e4)
        np.testing.assert_allclose(np.linalg.norm(qm), np.linalg.norm(q), rtol=1e-12)
        if (m, n) == (3, 1):
            ref = float(np.sum(qm * kn))
        np.testing.assert_allclose(np.sum(qm * kn), ref, rtol=1e-9)
    np.testing.assert_allclose(nm.rope(q, np.array([0]), 1e4), q)


def test_rmsnorm_softmax_silu_closed_forms():
    x = np.array([3.0, -4.0])
    np.testing.assert_allclose(nm.rmsnorm(x, np.array([2.0, 1.0]), 0.0), [2 * 3 / np.sqrt(12.5), -4 / np.sqrt(12.5)])
    np.testing.assert_allclose(nm.softmax(np.array([0.0, np.log(3.0)])), [0.25, 0.75])
    np.testing.assert_allclose(nm.silu(np.array([0.0, 1.0])), [0.0, 1 / (1 + np.exp(-1.0))])


def test_kv_rounding_is_the_only_effect_of_kv_bf16():
    shape = SHAPES["mha"]
    w = W.make_weights(shape, seed=3)
    prompt = W.make_prompt(shape.vocab, 6, seed=2)
    a, b = Decoder(LoopedLM(shape, w, kv_bf16=True)), Decoder(LoopedLM(shape, w, kv_bf16=False))
    a.prefill(prompt, 2), b.prefill(prompt, 2)
    Ka, Kb = a.K[1][0][:6], b.K[1][0][:6]
    np.testing.assert_array_equal(Ka, nm.round_bf16(Kb))          # layer 0, recurrence 1: same inputs
    assert np.abs(a.first_logits - b.first_logits).max() < 5e-3
