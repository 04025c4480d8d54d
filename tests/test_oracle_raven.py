"""Pins for the Raven-style layout in the oracle (Sec. 3.1: P and C hold transformer blocks; App. B "KV Cache Management":
prelude cache, one coda cache per readout depth): the cached, branch-wise path must equal a cache-free forward of the
whole prefix written with torch float64 library routines, at the final depth AND at the proposal depths, and the greedy
LoopSpec stream must be the vanilla stream.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as W
from oracle import depths as dp
from oracle.loopspec import Decoder
from oracle.model import LoopedLM


def torch_raven_forward(shape, w, ids, n_rec):
    """Cache-free: embedding -> prelude blocks -> n_rec x (adapter on [state; prelude output] -> recurrent blocks) ->
    coda blocks -> final norm -> lm_head.  Returns logits [n, V] (every position read out at depth n_rec)."""
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    n = len(ids)
    d, nq, nkv = shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    inv = shape.rope_theta ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    rot = torch.polar(torch.ones(n, d // 2, dtype=torch.float64), torch.arange(n, dtype=torch.float64)[:, None] * inv)

    def rms(v, g):
        return v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * t(g)

    def rotary(v):
        c = torch.complex(v[..., : d // 2], v[..., d // 2:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    def blocks(x, prefix, count):
        for l in range(count):
            g = lambda k: w[f"{prefix}.{l}.{k}"]
            y = rms(x, g("norm1")) @ t(g("wqkv")).T
            q = rotary(y[:, : nq * d].reshape(n, nq, d)).transpose(0, 1)
            k = rotary(y[:, nq * d:(nq + nkv) * d].reshape(n, nkv, d)).transpose(0, 1).repeat_interleave(nq // nkv, dim=0)
            v = y[:, (nq + nkv) * d:].reshape(n, nkv, d).transpose(0, 1).repeat_interleave(nq // nkv, dim=0)
            a = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=True)[0]
            x = x + a.transpose(0, 1).reshape(n, nq * d) @ t(g("wo")).T
            gu = rms(x, g("norm2")) @ t(g("wgateup")).T
            x = x + (F.silu(gu[:, : shape.ffn]) * gu[:, shape.ffn:]) @ t(g("wdown")).T
        return x

    e = blocks(t(w["embed"])[torch.tensor(np.asarray(ids), dtype=torch.long)], "prelude", shape.n_prelude)
    s = e
    for _ in range(n_rec):
        s = blocks(torch.cat([s, e], dim=1) @ t(w["adapter"]).T, "layers", shape.n_recurrent)
    x = blocks(s, "coda", shape.n_coda)
    head = w["embed"] if shape.tied else w["lm_head"]
    return (rms(x, w["final_norm"]) @ t(head).T).numpy()


SHAPE = W.CONFIGS["tiny"].with_(vocab=64, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=80, R=4, tied=False,
                                n_recurrent=2, n_prelude=2, n_coda=1, std=0.2)


def test_vanilla_equals_cache_free_forward():
    w = W.make_weights(SHAPE, seed=3, gain_jitter=0.1)
    model = LoopedLM(SHAPE, w, kv_bf16=False)
    prompt = W.make_prompt(SHAPE.vocab, 7, seed=5)
    dec = Decoder(model)
    dec.prefill(prompt, 6)
    toks, logits = dec.vanilla(5, keep_logits=True)
    full = torch_raven_forward(SHAPE, w, dec.ids[:-1], SHAPE.R)
    np.testing.assert_allclose(dec.first_logits, full[len(prompt) - 1], rtol=0, atol=1e-10)
    for i, z in enumerate(logits):
        np.testing.assert_allclose(z, full[len(prompt) + i], rtol=0, atol=1e-10)


@pytest.mark.parametrize("d1,d2", [(1, 2), (1, 3), (2, 0)])
def test_loopspec_readouts_equal_cache_free_forward_at_their_depth(d1, d2):
    """Every readout of the surviving root branch - at d1, at d2 and the verified ones at R - equals the cache-free forward
    of its prefix with that many recurrences (so the coda cache of each readout depth holds exactly the earlier
    positions' states AT THAT DEPTH), and the greedy stream is the vanilla one."""
    w = W.make_weights(SHAPE, seed=4, gain_jitter=0.1)
    model = LoopedLM(SHAPE, w, kv_bf16=False)
    prompt = W.make_prompt(SHAPE.vocab, 6, seed=6)
    van = Decoder(model)
    van.prefill(prompt, 16)
    ref = van.vanilla(12)
    dec = Decoder(model)
    dec.prefill(prompt, 16, depths=(d1, d2))
    seen, inner = [], dec._readout_logits

    def recording(b, depth):      # every readout with the full prefix of its branch (committed ids + uncommitted chain)
        chain, a = [], b
        while a is not None and a.parent is not None:
            chain.append(a.token)
            a = a.parent
        z = inner(b, depth)
        seen.append((dec.ids[: a.pos + 1] + chain[::-1], depth, z))
        return z
    dec._readout_logits = recording
    assert dec.loopspec(12, d1, d2, keep_logits=True) == ref
    n0 = len(prompt)
    full_R = torch_raven_forward(SHAPE, w, dec.ids[:-1], SHAPE.R)
    for i, z in enumerate(dec.verify_logits):
        np.testing.assert_allclose(z, full_R[n0 + i], rtol=0, atol=1e-10)
    assert len(seen) >= 12 and {dep for _, dep, _ in seen} == {d for d in (d1, d2, SHAPE.R) if d}
    for ids, depth, z in seen[:: max(1, len(seen) // 24)]:      # a spread of readouts, speculative branches included
        np.testing.assert_allclose(z, torch_raven_forward(SHAPE, w, ids, depth)[-1], rtol=0, atol=1e-10)
    st = dec.stats
    cost = {1: d1, 2: d2, 3: SHAPE.R}
    steps = [c["step"] for c in dec.commits]
    assert steps[0] == SHAPE.R and list(np.diff(steps)) == [cost[c["source"]] for c in dec.commits[:-1]]
    assert st["rows_max"] <= dp.max_branches(SHAPE.R, d1, d2)


@pytest.mark.parametrize("name,pairs", [("tiny_raven_r4", [(1, 2), (1, 3), (2, 0)]), ("tiny_raven", [(2, 8), (4, 8), (2, 4)])])
def test_greedy_and_sampled_runs_on_the_test_shapes(name, pairs):
    shape = W.CONFIGS[name]
    model = LoopedLM(shape, W.make_weights(shape))
    prompt = W.make_prompt(shape.vocab, 10)
    van = Decoder(model)
    van.prefill(prompt, 20)
    ref = van.vanilla(14)
    for d1, d2 in pairs:
        dec = Decoder(model)
        dec.prefill(prompt, 20, depths=(d1, d2))
        assert dec.loopspec(14, d1, d2) == ref, (d1, d2)
        assert dec.stats["rows_max"] <= dp.max_branches(shape.R, d1, d2)
    outs = []
    for _ in range(2):
        dec = Decoder(model, temperature=1.0, seed=3)
        dec.prefill(prompt, 20, depths=pairs[0])
        outs.append(dec.loopspec(14, *pairs[0]))
    assert outs[0] == outs[1]
