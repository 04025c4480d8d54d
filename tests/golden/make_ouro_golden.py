"""Writes tests/golden/ouro_1p4b_oracle.json: what the float64 oracle decodes on the Ouro-1.4B-shaped model
(the headline workload: prompt 512, greedy, (d1, d2) = (1, 2), gate on) for the first tokens of the run, the same
with temperature-1 sampling, and the same with the paper's sampling setting (temperature 1, top-p 0.7).  Calls only
`oracle/` and the seeded input generators.  Takes ~15 minutes and ~20 GB.  Runs already in the file are kept
(they are deterministic); pass --force to recompute them.

    python tests/golden/make_ouro_golden.py [n_tokens] [--force]
"""
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as W  # noqa: E402
from oracle.loopspec import Decoder  # noqa: E402
from oracle.model import LoopedLM  # noqa: E402


def main():
    args = [a for a in sys.argv[1:] if not a.startswith("--")]
    n_tokens = int(args[0]) if args else 24
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "ouro_1p4b_oracle.json")
    old = {}
    if os.path.exists(path) and "--force" not in sys.argv:
        with open(path) as f:
            old = json.load(f)
        if old.get("n_tokens") != n_tokens:
            old = {}
    wl = W.WORKLOADS["ouro_1p4b"]
    shape = W.CONFIGS[wl.model]
    t0 = time.time()
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed)
    out = {"workload": "ouro_1p4b", "prompt_len": wl.prompt_len, "n_tokens": n_tokens, "d1": wl.d1, "d2": wl.d2,
           "written_by": "tests/golden/make_ouro_golden.py (oracle only)", "runs": {}}
    probe = [0, 1, 17, 4095, 20000, 49151]
    for name, T, seed, top_p in (("greedy", 0.0, wl.sample_seed, 1.0), ("sampled_T1", 1.0, wl.sample_seed, 1.0),
                                 ("sampled_T1_top_p", 1.0, wl.sample_seed, 0.7)):
        if name in old.get("runs", {}):
            out["runs"][name] = old["runs"][name]
            continue
        dec = Decoder(model, temperature=T, seed=seed, top_p=top_p)
        first = dec.prefill(prompt, n_tokens + 4)
        toks = dec.loopspec(n_tokens, wl.d1, wl.d2, gate=wl.gate, keep_logits=True)
        out["runs"][name] = {
            "temperature": T, "top_p": top_p, "seed": seed, "first_token": first, "tokens": toks,
            "commits": [[c["source"], c["gate_open"], c["step"]] for c in dec.commits],
            "rows_per_step": dec.rows_per_step, "stats": {k: (float(v) if k == "gamma" else int(v)) for k, v in dec.stats.items()},
            "min_margin": min(e["margin"] for e in dec.log),
            "margins": [[e["kind"], e.get("pos", -1), float(e["margin"])] for e in dec.log],
            "first_logits_probe": {str(i): float(dec.first_logits[i]) for i in probe},
            "first_logits_argmax": int(np.argmax(dec.first_logits)),
            "last_verify_logits_probe": {str(i): float(dec.verify_logits[-1][i]) for i in probe},
        }
        print(name, "done", round(time.time() - t0), "s", "min margin", out["runs"][name]["min_margin"], flush=True)
    # vanilla tokens for the greedy run (losslessness at full size)
    if "vanilla_greedy_tokens" in old:
        out["vanilla_greedy_tokens"] = old["vanilla_greedy_tokens"]
    else:
        dec = Decoder(model, temperature=0.0)
        dec.prefill(prompt, n_tokens + 4)
        out["vanilla_greedy_tokens"] = dec.vanilla(n_tokens)
    with open(path, "w") as f:
        json.dump(out, f)
    print("written in", round(time.time() - t0), "s")


if __name__ == "__main__":
    main()
