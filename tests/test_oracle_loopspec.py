"""Pins for the scheduler (Algorithm 1; Sec. 4.2-4.3; proof of Thm 2 for the commit gaps)."""
import numpy as np
import pytest

import workloads as W
from oracle import depths as dp
from oracle.loopspec import Decoder
from oracle.model import LoopedLM

R = 4


def build(name, **kw):
    shape = W.CONFIGS[name].with_(**kw)
    return shape, LoopedLM(shape, W.make_weights(shape))


@pytest.fixture(scope="module")
def models():
    # high acceptance (tied, collapses to a repeated token) and low acceptance (untied)
    return {"tiny": build("tiny"), "tiny_untied": build("tiny", tied=False),
            "tiny_weak": build("tiny", tied=False, out_scale=0.02)}


@pytest.mark.parametrize("name", ["tiny", "tiny_untied", "tiny_weak"])
def test_greedy_loopspec_equals_vanilla_for_every_admissible_depth_pair(models, name):
    """North-star check (a): the greedy LoopSpec stream is the vanilla all-R stream, and the
    verified depth-R logits are the vanilla logits."""
    shape, model = models[name]
    prompt = W.make_prompt(shape.vocab, 16)
    n = 40
    van = Decoder(model)
    van.prefill(prompt, n)
    ref, ref_logits = van.vanilla(n, keep_logits=True)
    seen_sources = set()
    for d1, d2 in [(1, 0), (2, 0), (3, 0)] + dp.admissible_pairs(R) + [(2, 3)]:
        for gate in ([True, False] if d2 else [True]):
            dec = Decoder(model)
            assert dec.prefill(prompt, n) == van.ids[len(prompt)]
            out = dec.loopspec(n, d1, d2, gate=gate, keep_logits=True)
            assert out == ref, (name, d1, d2, gate)
            for a, b in zip(dec.verify_logits, ref_logits):
                np.testing.assert_allclose(a, b, rtol=0, atol=1e-10)
            st = dec.stats
            # commit gaps: d1 after an accepted first proposal, d2 after a second, R after a restart
            steps = [c["step"] for c in dec.commits]
            gaps = np.diff(steps)
            cost = {1: d1, 2: d2, 3: R}
            assert steps[0] == R
            assert list(gaps) == [cost[c["source"]] for c in dec.commits[:-1]]
            assert st["n_accept1"] + st["n_accept2"] + st["n_restart"] == n
            assert st["gamma"] <= R / d1 + 1e-12
            assert st["rows_max"] <= dp.max_branches(R, d1, d2) or d2 % d1 or R % d1
            seen_sources |= {c["source"] for c in dec.commits}
    if name == "tiny_untied":
        assert seen_sources == {1, 2, 3} or seen_sources == {2, 3}


@pytest.mark.parametrize("name,pairs", [("tiny_r8", [(1, 2), (1, 4), (2, 4), (2, 6), (4, 0)]),
                                        ("tiny_r16", [(2, 4), (2, 8), (4, 12), (8, 0)])])
def test_deeper_loops_greedy_equals_vanilla_and_rows_stay_under_the_bound(name, pairs):
    """Algorithm 1 for R = 8 and 16 (the Raven-style models loop 32 times): the greedy stream is the vanilla one, commit
    gaps are d1 / d2 / R, and the rows in flight never exceed the branch bound of Sec. 4.3."""
    shape, model = build(name)
    Rn = shape.R
    prompt = W.make_prompt(shape.vocab, 12)
    n = 24
    van = Decoder(model)
    van.prefill(prompt, n)
    ref = van.vanilla(n)
    for d1, d2 in pairs:
        dec = Decoder(model)
        dec.prefill(prompt, n)
        assert dec.loopspec(n, d1, d2) == ref, (name, d1, d2)
        steps = [c["step"] for c in dec.commits]
        cost = {1: d1, 2: d2, 3: Rn}
        assert steps[0] == Rn
        assert list(np.diff(steps)) == [cost[c["source"]] for c in dec.commits[:-1]]
        assert dec.stats["rows_max"] <= dp.max_branches(Rn, d1, d2)


def test_gamma_attains_R_over_d1_when_everything_is_accepted(models):
    shape, model = models["tiny"]
    dec = Decoder(model)
    dec.prefill(W.make_prompt(shape.vocab, 16), 64)
    dec.loopspec(64, 1)
    assert dec.stats["n_accept1"] == 64 and dec.stats["gamma"] == R


def test_sampled_loopspec_is_reproducible_and_self_consistent(models):
    shape, model = models["tiny_untied"]
    prompt = W.make_prompt(shape.vocab, 12)
    outs = []
    for _ in range(2):
        dec = Decoder(model, temperature=1.0, seed=2)
        dec.prefill(prompt, 30)
        outs.append(dec.loopspec(30, 1, 2))
    assert outs[0] == outs[1]
    kinds = {e["kind"] for e in dec.log}
    assert {"draft1", "gate", "accept1"} <= kinds
    other = Decoder(model, temperature=1.0, seed=3)
    other.prefill(prompt, 30)
    assert other.loopspec(30, 1, 2) != outs[0]


def test_sampled_loopspec_matches_vanilla_in_distribution(models):
    """Losslessness under sampling (Sec. 3.2): the first decoded token after the prefill token,
    over many seeds, follows the vanilla target distribution p_R(. | prompt, y0)."""
    shape = W.CONFIGS["tiny"].with_(vocab=16, hidden=32, n_q_heads=2, n_kv_heads=2, head_dim=16, ffn=48,
                                    tied=False, std=0.35)
    model = LoopedLM(shape, W.make_weights(shape, seed=9))
    prompt = W.make_prompt(shape.vocab, 4, seed=3)
    from scipy import stats
    base = Decoder(model, temperature=1.0, seed=0)
    y0 = base.prefill(prompt, 2)
    counts = np.zeros(shape.vocab)
    n, target = 1500, None
    srcs = np.zeros(4)
    for seed in range(n):
        dec = Decoder(model, temperature=1.0, seed=seed)
        dec.prefill(prompt, 2)
        if dec.ids[-1] != y0:            # condition on the same first token
            continue
        tok = dec.loopspec(1, 1, 2, keep_logits=True)[0]
        counts[tok] += 1
        srcs[dec.commits[0]["source"]] += 1
        target = dec.probs(dec.verify_logits[0])
    assert counts.sum() > 100 and srcs[1] > 0 and srcs[2] + srcs[3] > 0
    keep = target * counts.sum() > 5
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(target[keep], target[~keep].sum()) * counts.sum()
    if exp[-1] == 0:
        obs, exp = obs[:-1], exp[:-1]
    assert stats.chisquare(obs, exp).pvalue > 1e-3


def test_masked_second_proposal_keeps_greedy_lossless_and_candidates_distinct(models):
    """Second-proposal ablation (Sec. 6): with the first candidate masked out and the gate off, every branch gets a
    second candidate different from the first; greedy output still equals vanilla, and more tokens are accepted
    from second proposals than without the mask."""
    shape, model = models["tiny_untied"]
    prompt = W.make_prompt(shape.vocab, 12)
    van = Decoder(model)
    van.prefill(prompt, 40)
    want = van.vanilla(40)
    runs = {}
    for mask in (False, True):
        dec = Decoder(model)
        dec.prefill(prompt, 40)
        assert dec.loopspec(40, 1, 2, gate=False, mask_first=mask) == want
        runs[mask] = dec
    d1_at = {}
    for e in runs[True].log:
        if e["kind"] == "draft1":
            d1_at[e["pos"]] = e["token"]
        if e["kind"] == "draft2":
            assert e["token"] != d1_at[e["pos"]]
    assert runs[True].stats["n_accept2"] >= runs[False].stats["n_accept2"]
    # sampled: self-consistent and reproducible
    outs = []
    for _ in range(2):
        dec = Decoder(model, temperature=1.0, seed=5)
        dec.prefill(prompt, 30)
        outs.append(dec.loopspec(30, 1, 2, gate=False, mask_first=True))
    assert outs[0] == outs[1]


def test_filtered_sampling_is_lossless_in_distribution_and_stays_in_the_nucleus(models):
    """With top-k / top-p inside C (Sec. 3.1) the target is the filtered p_R: every committed token lies in its
    support, and the first decoded token over many seeds follows it."""
    shape = W.CONFIGS["tiny"].with_(vocab=16, hidden=32, n_q_heads=2, n_kv_heads=2, head_dim=16, ffn=48,
                                    tied=False, std=0.35)
    model = LoopedLM(shape, W.make_weights(shape, seed=9))
    prompt = W.make_prompt(shape.vocab, 4, seed=3)
    from scipy import stats
    kw = dict(temperature=1.0, top_k=12, top_p=0.8)
    base = Decoder(model, seed=0, **kw)
    y0 = base.prefill(prompt, 2)
    counts, target = np.zeros(shape.vocab), None
    for seed in range(1200):
        dec = Decoder(model, seed=seed, **kw)
        dec.prefill(prompt, 2)
        if dec.ids[-1] != y0:
            continue
        tok = dec.loopspec(1, 1, 2, keep_logits=True)[0]
        counts[tok] += 1
        target = dec.probs(dec.verify_logits[0])
    assert counts.sum() > 100
    assert 0 < np.count_nonzero(target) < shape.vocab          # the filter really cuts
    assert counts[target == 0].sum() == 0                      # nothing outside the nucleus is ever committed
    keep = target * counts.sum() > 5
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(target[keep], target[~keep].sum()) * counts.sum()
    if exp[-1] == 0:
        obs, exp = obs[:-1], exp[:-1]
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # a longer run: reproducible, and equal to the unfiltered run only if the filters are off
    a = Decoder(model, seed=5, **kw); a.prefill(prompt, 24)
    b = Decoder(model, seed=5, **kw); b.prefill(prompt, 24)
    assert a.loopspec(24, 1, 2) == b.loopspec(24, 1, 2)
    assert any(e["kind"] == "filter" for e in a.log)


class ScriptedModel:
    """A stub 'model' whose depth-R prediction for prefix ending in token t is t + 1 and whose early
    drafts are wrong exactly for the tokens listed in `bad_first` / `bad_second`."""

    class s:
        R = 4
        n_recurrent = 0
        n_kv_heads = 1
        head_dim = 2

    V = 64

    def __init__(self, bad_first=(), good_second=()):
        self.bad_first, self.good_second = set(bad_first), set(good_second)

    def embed_tokens(self, ids):
        return np.array([[float(t), 0.0] for t in ids])

    def advance_rows(self, X, pos, prefix_kv, E=None):
        X = np.array(X, dtype=np.float64)
        X[:, 1] += 1
        return X, [[] for _ in pos]

    def logits(self, x):
        t, depth = int(x[0]), int(x[1])
        z = np.zeros(self.V)
        guess = t + 1
        if depth == 1 and t in self.bad_first:
            guess = t + 30
        if depth in (2, 3) and t in self.bad_first and t not in self.good_second:
            guess = t + 31
        z[guess % self.V] = 1.0
        return z


def run_scripted(model, n, d1, d2=0):
    dec = Decoder(model)
    dec.ids = [0]
    dec._alloc(4)
    dec.loopspec(n, d1, d2)
    return dec


def test_timeline_single_proposal_R4_d1_1():
    """R = 4, d1 = 1: y1, y2 accepted, y3 rejected and resampled, y4 accepted (Fig. 1b pattern).
    Commits land at steps 4, 5, 6, 10 and the batch sizes are 1,2,3,4,4,4,1,2,3,4."""
    dec = run_scripted(ScriptedModel(bad_first={2}), 4, 1)
    assert dec.ids == [0, 1, 2, 3, 4]
    assert [c["step"] for c in dec.commits] == [4, 5, 6, 10]
    assert [c["source"] for c in dec.commits] == [1, 1, 3, 1]
    assert dec.rows_per_step == [1, 2, 3, 4, 4, 4, 1, 2, 3, 4]
    # gamma by hand (Sec. 6 "Implementation and Metrics"): 4 tokens x R = 16 recurrences' worth of output over
    # 3 first-proposal commits x d1 = 3 plus one restart x R = 4
    assert dec.stats["gamma"] == pytest.approx(16 / 7, abs=1e-15)
    assert (dec.stats["n_accept1"], dec.stats["n_accept2"], dec.stats["n_restart"]) == (3, 0, 1)


def test_timeline_second_proposal_saves_d2_steps():
    """With (d1, d2) = (1, 2): when the first draft of y3 is wrong but the depth-2 readout is right,
    the fallback child is kept and the next commit comes d2 = 2 steps later instead of R = 4 (Sec. 4.3)."""
    dec = run_scripted(ScriptedModel(bad_first={2}, good_second={2}), 5, 1, 2)
    assert dec.ids == [0, 1, 2, 3, 4, 5]
    assert [c["source"] for c in dec.commits] == [1, 1, 2, 1, 1]
    assert [c["step"] for c in dec.commits] == [4, 5, 6, 8, 9]
    assert [c["gate_open"] for c in dec.commits] == [0, 0, 1, 0, 0]
    # gamma by hand: 5 x 4 over 4 x d1 + 1 x d2 = 6; a second-proposal commit costs d2, not R (a formula with d2 and R
    # exchanged would give 20 / 8 here)
    assert dec.stats["gamma"] == pytest.approx(20 / 6, abs=1e-15)
    # both candidates wrong: restart, next commit R steps later
    dec = run_scripted(ScriptedModel(bad_first={2}), 4, 1, 2)
    assert [c["source"] for c in dec.commits] == [1, 1, 3, 1]
    assert [c["step"] for c in dec.commits] == [4, 5, 6, 10]
    assert dec.stats["gamma"] == pytest.approx(16 / 7, abs=1e-15)
    # R = 8 with (2, 4): every first draft right -> gamma = R / d1 = 4; the depth pair enters only through the costs
    class Deep(ScriptedModel):
        class s(ScriptedModel.s):
            R = 8

        def logits(self, x):
            t, depth = int(x[0]), int(x[1])
            z = np.zeros(self.V)
            wrong = t in self.bad_first and (depth == 2 or (depth == 4 and t not in self.good_second))
            z[(t + (30 if wrong else 1)) % self.V] = 1.0
            return z
    dec = run_scripted(Deep(bad_first={1, 3}, good_second={3}), 6, 2, 4)
    assert [c["source"] for c in dec.commits] == [1, 3, 1, 2, 1, 1]
    assert [c["step"] for c in dec.commits] == [8, 10, 18, 20, 24, 26]
    assert dec.stats["gamma"] == pytest.approx(6 * 8 / (4 * 2 + 1 * 4 + 1 * 8), abs=1e-15)


def test_tv_profile_of_a_verification_by_hand():
    """Sec. 4.1's empirical profile as logged at a verification: TV(p_d1, p_R) and TV(p_d2, p_R) for hand-made
    three-token distributions (0.5 x the L1 distance: 0.3 and 0.1)."""
    from oracle.loopspec import Branch, Record
    dec = Decoder(model=None, temperature=1.0, seed=4)
    p = np.array([0.5, 0.3, 0.2])
    q1 = np.array([0.2, 0.3, 0.5])
    q2t = np.array([0.4, 0.4, 0.2])
    b = Branch(parent=None, token=0, pos=5, H=None)
    b.records = [Record(2, q1, None), Record(0, q2t, None)]
    b.q2_logits = np.log(q2t) + 0.7          # any shift: C normalises
    tok, child, source = dec._verify(b, np.log(p) - 1.3)
    assert len(dec.tv_log) == 1
    tv1, tv2 = dec.tv_log[0]
    assert tv1 == pytest.approx(0.3, abs=1e-12) and tv2 == pytest.approx(0.1, abs=1e-12)
    # without a second record only the first distance is logged; under greedy decoding nothing is
    b.records = b.records[:1]
    dec._verify(b, np.log(p))
    assert dec.tv_log[1][0] == pytest.approx(0.3, abs=1e-12) and dec.tv_log[1][1] is None
    g = Decoder(model=None, temperature=0.0)
    g._verify(b, np.log(p))
    assert g.tv_log == []


def test_branch_census_reaches_the_bound_with_the_gate_forced_open():
    """Every branch forks at d1 and d2 (gate=False): 7 rows at the step the root reaches R for (4,1,2)."""
    dec = Decoder(ScriptedModel())
    dec.ids = [0]
    dec._alloc(4)
    dec.loopspec(6, 1, 2, gate=False)
    assert dec.rows_per_step[:4] == [1, 2, 4, 7]
    assert max(dec.rows_per_step) == dp.max_branches(4, 1, 2) == 7
    assert dec.ids == list(range(7))
