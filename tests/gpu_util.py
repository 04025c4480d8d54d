"""Helpers shared by the GPU parity tests: build the oracle run and the CUDA context for one case."""
import functools

import numpy as np

import workloads as W
from oracle.loopspec import Decoder
from oracle.model import LoopedLM


@functools.lru_cache(maxsize=None)
def np_weights(name, seed=0, gain_jitter=0.0):
    return W.make_weights(W.CONFIGS[name], seed=seed, gain_jitter=gain_jitter)


@functools.lru_cache(maxsize=None)
def oracle_model(name, seed=0, gain_jitter=0.0):
    return LoopedLM(W.CONFIGS[name], np_weights(name, seed, gain_jitter))


@functools.lru_cache(maxsize=None)
def oracle_run(name, n_prompt, n_decode, d1, d2, T=0.0, seed=2, gate=True, residual_q2=True, prompt_seed=1, seq=0,
               wseed=0, gain_jitter=0.0, vanilla=False, top_k=0, top_p=1.0, mask_first=False):
    shape = W.CONFIGS[name]
    dec = Decoder(oracle_model(name, wseed, gain_jitter), temperature=T, seed=seed, seq=seq, top_k=top_k, top_p=top_p)
    prompt = W.make_prompt(shape.vocab, n_prompt, seed=prompt_seed, seq=seq)
    first = dec.prefill(prompt, n_decode, depths=None if vanilla else (d1, d2))
    if vanilla:
        out, logits = dec.vanilla(n_decode, keep_logits=True)
        dec.verify_logits = logits
    else:
        out = dec.loopspec(n_decode, d1, d2, gate=gate, residual_q2=residual_q2, keep_logits=True,
                           mask_first=mask_first)
    return dict(prompt=prompt, first=first, tokens=out, dec=dec)


@functools.lru_cache(maxsize=None)
def gpu_weights(name, seed=0, gain_jitter=0.0):
    import paper_2609_17184_b200 as ls
    return ls.upload_weights(W.CONFIGS[name], np_weights(name, seed, gain_jitter))


def make_ctx(name, d1, d2, T=0.0, seed=2, gate=True, residual_q2=True, max_seqs=1, max_ctx=256, wseed=0, gain_jitter=0.0,
             **kw):
    import paper_2609_17184_b200 as ls
    return ls.LoopSpec(W.CONFIGS[name], gpu_weights(name, wseed, gain_jitter), d1=d1, d2=d2, temperature=T, seed=seed,
                       gate=gate, residual_q2=residual_q2, max_seqs=max_seqs, max_ctx=max_ctx, **kw)


def min_margin(dec):
    return min(e["margin"] for e in dec.log)


COMMIT_KEYS = ("token", "source", "accepted1", "accepted2", "gate_open", "step")


def assert_same_run(ctx, ref, n_decode, seq=0, logit_atol=3e-2, logit_rtol=2e-2):
    """The CUDA context (already decoded) against an oracle run: tokens, commit records, statistics, logits."""
    dec = ref["dec"]
    commits = ctx.commits(seq)
    got = [c["token"] for c in commits]
    assert got == ref["tokens"], (first_diff(got, ref["tokens"]), "oracle min margin", min_margin(dec))
    for g, o in zip(commits, dec.commits):
        assert tuple(g[k] for k in COMMIT_KEYS) == tuple(o[k] for k in COMMIT_KEYS), (g, o)
    z = ctx.debug_logits(seq, 0)
    zo = dec.verify_logits[-1]
    err = np.abs(z - zo)
    assert (err <= logit_atol + logit_rtol * np.abs(zo)).all(), err.max()
    # the proposal records Q_b of the surviving root branch: its depth-d1 and depth-d2 readouts, as stored for the
    # cascade verification still to come (Algorithm 1, Spawn / Verify), against the oracle's at the same tolerance
    root = next((b for b in getattr(dec, "active", []) if b.parent is None), None)
    if root is not None:
        for which, zq in ((1, root.q1_logits), (2, root.q2_logits)):
            if zq is None:
                continue
            eq = np.abs(ctx.debug_logits(seq, which) - zq)
            assert (eq <= logit_atol + logit_rtol * np.abs(zq)).all(), (which, eq.max())
            err = np.maximum(err, eq)
    return err.max()


def first_diff(a, b):
    for i, (x, y) in enumerate(zip(a, b)):
        if x != y:
            return i, x, y
    return None
