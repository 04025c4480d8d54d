"""Full-size parity on the Ouro-1.4B-shaped model (the headline workload: prompt 512, 512 greedy tokens), in the launch configuration bench.py times.

The oracle cannot decode 512 tokens of a 1.4B model in test time, so:
  * the first tokens of the run (greedy, temperature 1, temperature 1 with top-p 0.7) are compared with values the
    oracle computed once
    (tests/golden/ouro_1p4b_oracle.json, written by tests/golden/make_ouro_golden.py, which calls only oracle/);
  * the whole 512-token run is checked through properties that hold at any size: greedy LoopSpec == greedy
    vanilla decoding on the device, the commit-gap schedule, and the counters' identities.
"""
import json
import os

import numpy as np
import pytest

import workloads as W

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden", "ouro_1p4b_oracle.json")


@pytest.fixture(scope="module")
def setup():
    import paper_2609_17184_b200 as ls
    wl = W.WORKLOADS["ouro_1p4b"]
    shape = W.CONFIGS[wl.model]
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    return ls, wl, shape, weights, prompt, json.load(open(GOLD))


def make(setup, T, top_p=1.0):
    ls, wl, shape, weights, prompt, gold = setup
    return ls.LoopSpec(shape, weights, d1=wl.d1, d2=wl.d2, temperature=T, seed=wl.sample_seed, gate=wl.gate, max_seqs=1,
                       max_ctx=wl.prompt_len + wl.decode_len + 16, max_prefill_rows=64, top_p=top_p)


@pytest.mark.parametrize("run", ["greedy", "sampled_T1", "sampled_T1_top_p"])
def test_first_tokens_match_the_oracle(setup, run):
    ls, wl, shape, weights, prompt, gold = setup
    g = gold["runs"][run]
    n = gold["n_tokens"]
    ctx = make(setup, g["temperature"], g.get("top_p", 1.0))
    assert ctx.prefill(prompt) == g["first_token"]
    z = ctx.debug_logits(0, 0)
    assert int(np.argmax(z)) == g["first_logits_argmax"]
    for i, v in g["first_logits_probe"].items():
        assert abs(z[int(i)] - v) <= 3e-2 + 2e-2 * abs(v)
        assert abs(z[int(i)] - v) < 5e-3
    out = ctx.decode(n)[0].tolist()
    decisions = sorted(m[2] for m in g["margins"] if m[0] != "filter")
    assert out == g["tokens"], ("oracle's closest decisions (nucleus edges aside)", decisions[:3], "closest of all", g["min_margin"])
    commits = ctx.commits(0)
    assert [[c["source"], c["gate_open"], c["step"]] for c in commits] == g["commits"]
    assert ctx.row_trace().tolist() == g["rows_per_step"]
    st = ctx.stats()
    for k, v in g["stats"].items():
        if k != "gamma":
            assert st[k] == v, k
    z = ctx.debug_logits(0, 0)
    for i, v in g["last_verify_logits_probe"].items():
        assert abs(z[int(i)] - v) < 5e-3
    if run == "greedy":
        ctx.prefill(prompt)
        assert ctx.vanilla_decode(n)[0].tolist() == gold["vanilla_greedy_tokens"] == g["tokens"]
    ctx.close()


def test_full_run_properties(setup):
    ls, wl, shape, weights, prompt, gold = setup
    n, R = wl.decode_len, shape.R
    ctx = make(setup, 0.0)
    ctx.prefill(prompt)
    out = ctx.decode(n)[0].tolist()
    commits, st, trace = ctx.commits(0), ctx.stats(), ctx.row_trace()
    assert out[: gold["n_tokens"]] == gold["runs"]["greedy"]["tokens"]
    # schedule: first commit after R passes, then d1 / d2 / R passes after a first / second / resampled commit
    cost = {1: wl.d1, 2: wl.d2, 3: R}
    steps = [c["step"] for c in commits]
    assert steps[0] == R and list(np.diff(steps)) == [cost[c["source"]] for c in commits[:-1]]
    assert st["n_decode"] == n == st["n_accept1"] + st["n_accept2"] + st["n_restart"]
    assert st["steps"] == steps[-1] == len(trace) and st["rows_total"] == int(trace.sum()) and st["rows_max"] == int(trace.max())
    assert st["rows_max"] <= ls.max_branches(R, wl.d1, wl.d2)
    den = st["n_accept1"] * wl.d1 + st["n_accept2"] * wl.d2 + st["n_restart"] * R
    assert abs(st["gamma"] - n * R / den) < 1e-12
    # losslessness at full size: the pipelined greedy stream is the vanilla all-R stream
    ctx.prefill(prompt)
    assert ctx.vanilla_decode(n)[0].tolist() == out
    # and the run is reproducible bit for bit (logits of the last verification)
    z1 = ctx.debug_logits(0, 0).copy()
    ctx.prefill(prompt)
    ctx.vanilla_decode(n)
    assert np.array_equal(z1.view(np.uint32), ctx.debug_logits(0, 0).view(np.uint32))
    ctx.close()


# ---- Ouro-2.6B shape: temperature 1 with rejection verification, depths from the closed form (Theorem 2) ---------------
GOLD_2P6B = os.path.join(os.path.dirname(__file__), "golden", "ouro_2p6b_oracle.json")


def test_ouro_2p6b_closed_form_run_matches_the_oracle():
    """48 shared layers, prompt 1024, T = 1.  The oracle decoded a few tokens the vanilla way while reading out every
    depth (TV profile of Sec. 4.1), fitted the envelope, took the admissible pair minimising Theorem 2's bound and ran
    LoopSpec with it (tests/golden/make_config_goldens.py).  The device repeats the same calls: the host-side fit and
    depth picker give the same pair from the oracle's profile, and tokens, commit records, row counts and logits agree."""
    import paper_2609_17184_b200 as ls
    g = json.load(open(GOLD_2P6B))
    wl = W.WORKLOADS["ouro_2p6b"]
    shape = W.CONFIGS[wl.model]
    alpha, beta = ls.fit_envelope(g["tv_profile"])
    assert abs(alpha - g["alpha"]) < 1e-9 and abs(beta - g["beta"]) < 1e-9
    d1s, d2s, d1, d2 = ls.pick_depths(alpha, beta, shape.R)
    assert (d1, d2) == (g["d1"], g["d2"]) and abs(d1s - g["d1_star"]) < 1e-5 and abs(d2s - g["d2_star"]) < 1e-5
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    ctx = ls.LoopSpec(shape, weights, d1=d1, d2=d2, temperature=g["temperature"], seed=g["seed"], gate=wl.gate, max_seqs=1,
                      max_ctx=wl.prompt_len + 64, max_prefill_rows=64)
    assert ctx.prefill(prompt) == g["first_token"]
    z = ctx.debug_logits(0, 0)
    assert int(np.argmax(z)) == g["first_logits_argmax"]
    for i, v in g["first_logits_probe"].items():
        assert abs(z[int(i)] - v) <= 3e-2 + 2e-2 * abs(v) and abs(z[int(i)] - v) < 5e-3
    n0, n = g["n_profile"], g["n_tokens"]
    assert ctx.vanilla_decode(n0)[0].tolist() == g["vanilla_tokens"]
    run = g["run"]
    assert ctx.decode(n)[0].tolist() == run["tokens"], ("oracle min margin", run["min_margin"])
    commits = ctx.commits(0)[n0:]
    assert [[c["source"], c["gate_open"], c["step"]] for c in commits] == run["commits"]
    assert ctx.row_trace().tolist() == run["rows_per_step"]
    st = ctx.stats()
    for k, v in run["stats"].items():
        if k != "gamma":
            assert st[k] == v, k
    assert abs(st["gamma"] - run["stats"]["gamma"]) < 1e-12
    z = ctx.debug_logits(0, 0)
    for i, v in run["last_verify_logits_probe"].items():
        assert abs(z[int(i)] - v) < 5e-3
    ctx.close()


# ---- KV-bound serving regime at reduced size: several long sequences, temperature 0.7, per-sequence rollback -----------
GOLD_KV = os.path.join(os.path.dirname(__file__), "golden", "kv_bound_small_oracle.json")


def test_kv_bound_regime_at_reduced_size_matches_the_oracle():
    """Two independent sequences with 2600-token prompts on the Ouro-1.4B shape (contexts beyond 40 attention chunks: the
    run-based attention kernel; passes of up to 14 rows), T = 0.7 with rejection verification: every sequence decodes the
    oracle's tokens with the oracle's accept / reject decisions, and exactly what it decodes alone (per-sequence
    rollback of the depth-indexed KV cache; a token's arithmetic does not depend on what shares the pass)."""
    import paper_2609_17184_b200 as ls
    g = json.load(open(GOLD_KV))
    shape = W.CONFIGS[g["model"]]
    wl = W.WORKLOADS["kv_bound"]
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    n, S = g["n_tokens"], g["n_seqs"]
    prompts = [W.make_prompt(shape.vocab, g["prompt_len"], seed=wl.prompt_seed, seq=s) for s in range(S)]
    kw = dict(d1=g["d1"], d2=g["d2"], temperature=g["temperature"], seed=g["seed"], gate=wl.gate,
              max_ctx=g["prompt_len"] + n + 16, max_prefill_rows=64)
    ctx = ls.LoopSpec(shape, weights, max_seqs=S, **kw)
    for s in range(S):
        assert ctx.prefill(prompts[s], seq=s) == g["seqs"][s]["first_token"]
    out = ctx.decode(n)
    logits = []
    for s in range(S):
        rec = g["seqs"][s]
        assert out[s].tolist() == rec["tokens"], (s, "oracle min margin", rec["min_margin"])
        src_gate = [[c["source"], c["gate_open"]] for c in ctx.commits(s)]
        assert src_gate == [c[:2] for c in rec["commits"]], s
        z = ctx.debug_logits(s, 0)
        for i, v in rec["last_verify_logits_probe"].items():
            assert abs(z[int(i)] - v) < 5e-3
        logits.append(z.copy())
    ctx.close()
    for s in range(S):      # alone, in slot s of a context of the same width: bit-identical logits
        alone = ls.LoopSpec(shape, weights, max_seqs=S, **kw)
        alone.prefill(prompts[s], seq=s)
        assert alone.decode(n)[s].tolist() == g["seqs"][s]["tokens"]
        assert [c["step"] for c in alone.commits(s)] == [c[2] for c in g["seqs"][s]["commits"]]
        assert np.array_equal(alone.debug_logits(s, 0).view(np.uint32), logits[s].view(np.uint32))
        alone.close()


# ---- Raven-style workload at full size (prelude / adapter / recurrent / coda blocks, R = 16, GQA 32:8 x 64, V = 128256) --------
GOLD_RAVEN = os.path.join(os.path.dirname(__file__), "golden", "raven_oracle.json")


def test_raven_style_workload_at_full_size_matches_the_oracle():
    """Prompt 256, greedy, (d1, d2) = (2, 8), in the launch configuration bench.py times (passes of up to 18 rows: the
    layers' GEMMs on the tcgen05 kernel, readout on the cluster kernel): first token, its logits, the first tokens of
    the run with their commit records and row counts, the last verified logits; and greedy LoopSpec == vanilla."""
    import paper_2609_17184_b200 as ls
    g = json.load(open(GOLD_RAVEN))
    wl = W.WORKLOADS["raven"]
    shape = W.CONFIGS[wl.model]
    assert (g["d1"], g["d2"], g["prompt_len"]) == (wl.d1, wl.d2, wl.prompt_len)
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    ctx = ls.LoopSpec(shape, weights, d1=wl.d1, d2=wl.d2, temperature=wl.temperature, seed=wl.sample_seed, gate=wl.gate, max_seqs=1,
                      max_ctx=wl.prompt_len + wl.decode_len + 16, max_prefill_rows=64)
    assert ctx.decode_paths()[0] == 1
    assert ctx.prefill(prompt) == g["first_token"]
    z = ctx.debug_logits(0, 0)
    assert int(np.argmax(z)) == g["first_logits_argmax"]
    for i, v in g["first_logits_probe"].items():
        assert abs(z[int(i)] - v) <= 3e-2 + 2e-2 * abs(v)
    run, n = g["run"], g["n_tokens"]
    out = ctx.decode(n)[0].tolist()
    decisions = sorted(m[2] for m in run["margins"] if m[0] != "filter")
    assert out == run["tokens"], ("oracle's closest decisions", decisions[:3])
    commits = ctx.commits(0)
    assert [[c["source"], c["gate_open"], c["step"]] for c in commits] == run["commits"]
    assert ctx.row_trace().tolist() == run["rows_per_step"]
    st = ctx.stats()
    for k, v in run["stats"].items():
        if k != "gamma":
            assert st[k] == v, k
    z = ctx.debug_logits(0, 0)
    for i, v in run["last_verify_logits_probe"].items():
        assert abs(z[int(i)] - v) <= 3e-2 + 2e-2 * abs(v)
    ctx.prefill(prompt)
    assert ctx.vanilla_decode(n)[0].tolist() == run["tokens"]
    ctx.close()
