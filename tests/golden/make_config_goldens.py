"""Writes the oracle's runs for two more of the benchmark's workloads (calls only `oracle/` and the seeded generators):

  ouro_2p6b_oracle.json   Ouro-2.6B shape (48 shared layers, R = 4), prompt 1024, temperature 1 with rejection-sampling
                          verification, proposal depths from the closed form of Theorem 2: the oracle first decodes a
                          few tokens the vanilla way and reads out every depth (the empirical TV profile of Sec. 4.1),
                          fits the envelope, takes the admissible pair minimising the bound, then runs LoopSpec with it.
  kv_bound_small_oracle.json  the KV-bound serving regime at reduced size: two independent sequences on the Ouro-1.4B
                          shape with 2600-token prompts (contexts beyond 40 attention chunks), temperature 0.7,
                          (d1, d2) = (1, 2): tokens, commit records and row counts per sequence.

  raven_oracle.json       the Raven-style workload at full size (2 prelude + 4 recurrent + 2 coda blocks, R = 16, prompt
                          256, greedy, (d1, d2) = (2, 8)): the first tokens with commit records, row counts and logit probes.

    python tests/golden/make_config_goldens.py 2p6b|kv|raven [--force]

Each takes tens of minutes and 12-25 GB of memory.
"""
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as W  # noqa: E402
from oracle import depths as dp  # noqa: E402
from oracle import numerics as nm  # noqa: E402
from oracle import sampling as sp  # noqa: E402
from oracle.loopspec import Decoder  # noqa: E402
from oracle.model import LoopedLM  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))
PROBE = [0, 1, 17, 4095, 20000, 49151]


def run_record(dec, toks, first=None):
    rec = {"tokens": toks, "commits": [[c["source"], c["gate_open"], c["step"]] for c in dec.commits],
           "rows_per_step": dec.rows_per_step,
           "stats": {k: (float(v) if k == "gamma" else int(v)) for k, v in dec.stats.items()},
           "min_margin": min(e["margin"] for e in dec.log),
           "margins": [[e["kind"], e.get("pos", -1), float(e["margin"])] for e in dec.log],
           "last_verify_logits_probe": {str(i): float(dec.verify_logits[-1][i]) for i in PROBE}}
    if first is not None:
        rec["first_token"] = first
        rec["first_logits_probe"] = {str(i): float(dec.first_logits[i]) for i in PROBE}
        rec["first_logits_argmax"] = int(np.argmax(dec.first_logits))
    return rec


def tv_profile_by_vanilla(dec, n_tokens):
    """Decode n_tokens the vanilla way (all R recurrences per token), reading out EVERY depth on the way: returns the
    tokens and the mean TV(p_r, p_R) for r = 1..R-1 (Sec. 4.1).  Mirrors Decoder.vanilla, with the extra readouts."""
    s = dec.m.s
    out, acc = [], np.zeros(s.R - 1)
    for _ in range(n_tokens):
        pos = len(dec.ids) - 1
        x = dec.m.embed_tokens([dec.ids[-1]])
        early = []
        for r in range(1, s.R + 1):
            x, own = dec.m.advance_rows(x, [pos], lambda i, l, r=r: (dec.K[r][l][:pos], dec.V[r][l][:pos]))
            dec._store_committed(r, pos, own[0])
            if r < s.R:
                early.append(nm.softmax(dec.m.logits(x[0]) / dec.T))
        z = dec.m.logits(x[0])
        p = nm.softmax(z / dec.T)
        acc += [0.5 * float(np.abs(q - p).sum()) for q in early]
        tok, margin = dec._sample_target(z, pos + 1, sp.VANILLA)
        dec.log.append(dict(kind="vanilla", pos=pos + 1, token=tok, margin=margin))
        dec.ids.append(tok)
        out.append(tok)
    return out, (acc / n_tokens).tolist()


def golden_2p6b(path):
    wl = W.WORKLOADS["ouro_2p6b"]
    shape = W.CONFIGS[wl.model]
    n_profile, n_tokens = 6, 16
    t0 = time.time()
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    dec = Decoder(model, temperature=wl.temperature, seed=wl.sample_seed)
    first = dec.prefill(prompt, n_profile + n_tokens + 4)
    print("prefill done", round(time.time() - t0), "s", flush=True)
    van, tv = tv_profile_by_vanilla(dec, n_profile)
    alpha, beta = dp.fit_envelope(tv)
    d1s, d2s = dp.optimal_depths(alpha, beta, shape.R)
    d1, d2 = dp.snap_depths(alpha, beta, shape.R)
    print("profile", tv, "alpha, beta", alpha, beta, "closed form", d1s, d2s, "pair", d1, d2, round(time.time() - t0), "s", flush=True)
    toks = dec.loopspec(n_tokens, d1, d2, gate=wl.gate, keep_logits=True)
    out = {"workload": "ouro_2p6b", "prompt_len": wl.prompt_len, "temperature": wl.temperature, "seed": wl.sample_seed,
           "written_by": "tests/golden/make_config_goldens.py (oracle only)",
           "first_token": first, "first_logits_probe": {str(i): float(dec.first_logits[i]) for i in PROBE},
           "first_logits_argmax": int(np.argmax(dec.first_logits)),
           "n_profile": n_profile, "vanilla_tokens": van, "tv_profile": tv, "alpha": alpha, "beta": beta,
           "d1_star": d1s, "d2_star": d2s, "d1": d1, "d2": d2, "n_tokens": n_tokens, "run": run_record(dec, toks)}
    with open(path, "w") as f:
        json.dump(out, f)
    print("written in", round(time.time() - t0), "s", flush=True)


def golden_kv(path):
    shape = W.CONFIGS["ouro_1p4b"]
    wl = W.WORKLOADS["kv_bound"]
    n_prompt, n_tokens, n_seqs = 2600, 8, 2
    t0 = time.time()
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    out = {"workload": "kv_bound at reduced size", "model": "ouro_1p4b", "prompt_len": n_prompt, "n_seqs": n_seqs,
           "temperature": wl.temperature, "seed": wl.sample_seed, "d1": wl.d1, "d2": wl.d2, "n_tokens": n_tokens,
           "written_by": "tests/golden/make_config_goldens.py (oracle only)", "seqs": []}
    for s in range(n_seqs):
        prompt = W.make_prompt(shape.vocab, n_prompt, seed=wl.prompt_seed, seq=s)
        dec = Decoder(model, temperature=wl.temperature, seed=wl.sample_seed, seq=s)
        first = dec.prefill(prompt, n_tokens + 4)
        print("seq", s, "prefill done", round(time.time() - t0), "s", flush=True)
        toks = dec.loopspec(n_tokens, wl.d1, wl.d2, gate=wl.gate, keep_logits=True)
        out["seqs"].append(run_record(dec, toks, first))
        print("seq", s, "done", round(time.time() - t0), "s", "min margin", out["seqs"][-1]["min_margin"], flush=True)
    with open(path, "w") as f:
        json.dump(out, f)
    print("written in", round(time.time() - t0), "s", flush=True)


def golden_raven(path):
    wl = W.WORKLOADS["raven"]
    shape = W.CONFIGS[wl.model]
    n_tokens = 12
    t0 = time.time()
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    dec = Decoder(model, temperature=wl.temperature, seed=wl.sample_seed)
    first = dec.prefill(prompt, n_tokens + 4, depths=(wl.d1, wl.d2))
    print("prefill done", round(time.time() - t0), "s", flush=True)
    toks = dec.loopspec(n_tokens, wl.d1, wl.d2, gate=wl.gate, keep_logits=True)
    probe = [i for i in PROBE if i < shape.vocab] + [shape.vocab - 1]
    rec = run_record(dec, toks)
    rec["last_verify_logits_probe"] = {str(i): float(dec.verify_logits[-1][i]) for i in probe}
    out = {"workload": "raven", "prompt_len": wl.prompt_len, "temperature": wl.temperature, "seed": wl.sample_seed,
           "d1": wl.d1, "d2": wl.d2, "written_by": "tests/golden/make_config_goldens.py (oracle only)",
           "first_token": first, "first_logits_probe": {str(i): float(dec.first_logits[i]) for i in probe},
           "first_logits_argmax": int(np.argmax(dec.first_logits)), "n_tokens": n_tokens, "run": rec}
    with open(path, "w") as f:
        json.dump(out, f)
    print("written in", round(time.time() - t0), "s", "min margin", rec["min_margin"], flush=True)


if __name__ == "__main__":
    which = [a for a in sys.argv[1:] if not a.startswith("--")]
    jobs = {"2p6b": ("ouro_2p6b_oracle.json", golden_2p6b), "kv": ("kv_bound_small_oracle.json", golden_kv),
            "raven": ("raven_oracle.json", golden_raven)}
    for w in which or list(jobs):
        name, fn = jobs[w]
        path = os.path.join(HERE, name)
        if os.path.exists(path) and "--force" not in sys.argv:
            print(name, "exists (pass --force to recompute)")
            continue
        fn(path)
