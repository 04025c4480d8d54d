"""Pins for the random draws and the rejection rule (Sec. 3.2 Eq. 2-4; Sec. 4.3; Thm 1; App. G)."""
import itertools

import numpy as np
import pytest
from scipy import stats

from oracle import sampling as sp
from oracle.loopspec import Branch, Decoder, Record


# ---- Philox4x32-10: known-answer vectors published with the Random123 library --------------
KAT = [
    ((0, 0, 0, 0), (0, 0), (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)),
    ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2, (0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD)),
    ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0),
     (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1)),
]


@pytest.mark.parametrize("ctr,key,out", KAT)
def test_philox_known_answers(ctr, key, out):
    got = tuple(int(x) for x in sp.philox4x32_10(ctr, key))
    assert got == out


def test_uniform_and_gumbel_ranges_and_moments():
    pos = np.arange(200000)
    u = sp.uniform(7, 0, pos, sp.ACCEPT1)
    assert u.min() > 0 and u.max() < 1
    assert abs(u.mean() - 0.5) < 3e-3 and abs(u.var() - 1 / 12) < 2e-3
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    g = sp.gumbel(7, 0, np.arange(20000), sp.DRAFT1, 10).ravel()
    assert abs(g.mean() - np.euler_gamma) < 1e-2 and abs(g.var() - np.pi ** 2 / 6) < 3e-2
    # different purposes / sequences / positions give different streams
    assert not np.allclose(u[:100], sp.uniform(7, 0, pos[:100], sp.ACCEPT2))
    assert not np.allclose(u[:100], sp.uniform(7, 1, pos[:100], sp.ACCEPT1))
    assert not np.allclose(u[:100], sp.uniform(8, 0, pos[:100], sp.ACCEPT1))
    # scalar and vector calls agree
    assert sp.uniform(7, 0, 5, sp.ACCEPT1) == u[5]


def test_residual_operator_definition():
    mu, nu = np.array([0.5, 0.3, 0.2]), np.array([0.2, 0.3, 0.5])
    np.testing.assert_allclose(sp.residual(mu, nu), [1.0, 0.0, 0.0])
    mu, nu = np.array([0.4, 0.4, 0.2]), np.array([0.1, 0.2, 0.7])
    np.testing.assert_allclose(sp.residual(mu, nu), [0.6, 0.4, 0.0])
    np.testing.assert_allclose(sp.residual(mu, mu), mu)          # no positive part: fall back to mu


def random_dist(rng, V, conc=1.0):
    return rng.dirichlet(np.full(V, conc))


def cascade_law(p, q1, q2t, gate=True, residual_q2=True, mask_first=False):
    """Exact output law of drafting + cascade verification, by enumeration over (x1, x2)."""
    V = len(p)
    law = np.zeros(V)
    rho1 = sp.residual(p, q1)
    q2_plain = sp.residual(q2t, q1) if residual_q2 else q2t
    p_rej1 = p_rej_both = 0.0
    for x1 in range(V):
        if q1[x1] == 0:
            continue
        a1 = sp.accept_prob(p, q1, x1)
        law[x1] += q1[x1] * a1
        rej = q1[x1] * (1 - a1)
        p_rej1 += rej
        if gate and not (q2t[x1] < q1[x1]):
            law += rej * rho1
            p_rej_both += rej
            continue
        q2 = sp.masked_second_proposal(q2t, q1, x1, residual_q2) if mask_first else q2_plain
        if q2 is None:                      # nothing left to propose: resample from the first residual
            law += rej * rho1
            p_rej_both += rej
            continue
        rho2 = sp.residual(rho1, q2)
        for x2 in range(V):
            if q2[x2] == 0:
                continue
            a2 = sp.accept_prob(rho1, q2, x2)
            law[x2] += rej * q2[x2] * a2
            law += rej * q2[x2] * (1 - a2) * rho2
            p_rej_both += rej * q2[x2] * (1 - a2)
    return law, p_rej1, p_rej_both


@pytest.mark.parametrize("V", [3, 5, 8])
@pytest.mark.parametrize("gate,residual_q2", [(True, True), (False, True), (False, False), (True, False)])
def test_cascade_is_lossless_by_enumeration(V, gate, residual_q2):
    rng = np.random.default_rng(V)
    for _ in range(20):
        p, q1, q2t = (random_dist(rng, V, c) for c in (0.7, 1.0, 0.8))
        law, _, _ = cascade_law(p, q1, q2t, gate, residual_q2)
        np.testing.assert_allclose(law, p, atol=1e-12)


def test_masked_second_proposal_definition_and_losslessness():
    """Second-proposal ablation (Sec. 6): masking the first candidate gives a distribution with no mass on it, in
    proportion to the unmasked proposal elsewhere; verification stays exact for it (any proposal is admissible)."""
    rng = np.random.default_rng(21)
    for V in (3, 6):
        for _ in range(20):
            p, q1, q2t = (random_dist(rng, V, c) for c in (0.7, 1.0, 0.8))
            for residual_q2 in (True, False):
                for gate in (True, False):
                    law, _, _ = cascade_law(p, q1, q2t, gate, residual_q2, mask_first=True)
                    np.testing.assert_allclose(law, p, atol=1e-12)
                x1 = int(rng.integers(V))
                q2 = sp.masked_second_proposal(q2t, q1, x1, residual_q2)
                plain = sp.residual(q2t, q1) if residual_q2 else q2t
                assert q2[x1] == 0 and abs(q2.sum() - 1) < 1e-12
                others = np.arange(V) != x1
                if plain[others].sum() > 0:
                    np.testing.assert_allclose(q2[others], plain[others] / plain[others].sum(), atol=1e-12)
    # degenerate cases: the residual sits on x1 alone -> q2~ without x1; q2~ sits on x1 alone -> no proposal
    q1 = np.array([0.5, 0.5, 0.0]); q2t = np.array([0.7, 0.3, 0.0])
    np.testing.assert_allclose(sp.masked_second_proposal(q2t, q1, 0), [0, 1, 0])
    assert sp.masked_second_proposal(np.array([1.0, 0, 0]), q1, 0) is None
    assert sp.masked_second_proposal(np.array([1.0, 0, 0]), q1, 0, residual_q2=False) is None


def tv(a, b):
    return 0.5 * np.abs(a - b).sum()


def test_acceptance_probability_is_one_minus_tv_and_theorem_1_bounds():
    rng = np.random.default_rng(11)
    for _ in range(200):
        V = int(rng.integers(3, 9))
        p, q1, q2t = (random_dist(rng, V, c) for c in (0.6, 1.0, 0.9))
        _, rej1, rej_both_gated = cascade_law(p, q1, q2t, gate=True)
        _, _, rej_both_open = cascade_law(p, q1, q2t, gate=False)
        eps2 = tv(q2t, p)
        assert abs((1 - rej1) - (1 - tv(q1, p))) < 1e-12           # Pr[accept] = 1 - TV (App. G)
        assert rej_both_open <= eps2 + 1e-12                        # Thm 1, no gate
        assert rej_both_gated <= 2 * eps2 + 1e-12                   # Thm 1, with gate


def test_open_gate_excludes_first_candidate_from_residual_proposal():
    rng = np.random.default_rng(5)
    for _ in range(100):
        q1, q2t = random_dist(rng, 6), random_dist(rng, 6)
        q2 = sp.residual(q2t, q1)
        for x1 in range(6):
            if q2t[x1] < q1[x1]:
                assert q2[x1] == 0.0


def vector_cascade(seed, p, q1, q2t, n, gate=True):
    """n independent drafts + verifications composed from the oracle's vectorised primitives."""
    V = len(p)
    pos = np.arange(n)
    x1, _ = sp.race(np.broadcast_to(q1, (n, V)), sp.gumbel(seed, 0, pos, sp.DRAFT1, V))
    q2 = sp.residual(q2t, q1)
    is_open = (q2t[x1] < q1[x1]) | (not gate)
    x2, _ = sp.race(np.broadcast_to(q2, (n, V)), sp.gumbel(seed, 0, pos, sp.DRAFT2, V))
    U1 = sp.uniform(seed, 0, pos, sp.ACCEPT1)
    U2 = sp.uniform(seed, 0, pos, sp.ACCEPT2)
    acc1 = U1 < np.minimum(1.0, p[x1] / q1[x1])
    rho1 = sp.residual(p, q1)
    acc2 = is_open & ~acc1 & (U2 < np.minimum(1.0, rho1[x2] / q2[x2]))
    rho2 = sp.residual(rho1, q2)
    g = sp.gumbel(seed, 0, pos, sp.RESAMPLE, V)
    r_open, _ = sp.race(np.broadcast_to(rho2, (n, V)), g)
    r_closed, _ = sp.race(np.broadcast_to(rho1, (n, V)), g)
    out = np.where(acc1, x1, np.where(acc2, x2, np.where(is_open, r_open, r_closed)))
    src = np.where(acc1, 1, np.where(acc2, 2, 3))
    return out, src, x1, x2, is_open


def test_rejection_sampling_reproduces_target_chi_square_1e6():
    """North-star check (b): 10^6 cascade draws on a 16-token vocabulary follow p_R."""
    rng = np.random.default_rng(2)
    V, n = 16, 1_000_000
    p, q1, q2t = random_dist(rng, V, 0.5), random_dist(rng, V, 0.8), random_dist(rng, V, 0.6)
    out, src, *_ = vector_cascade(1234, p, q1, q2t, n)
    counts = np.bincount(out, minlength=V)
    chi2, pval = stats.chisquare(counts, p * n)
    assert pval > 1e-3, (chi2, pval)
    law, rej1, rej_both = cascade_law(p, q1, q2t)
    assert abs((src != 1).mean() - rej1) < 4 * np.sqrt(rej1 * (1 - rej1) / n) + 1e-9
    assert abs((src == 3).mean() - rej_both) < 4 * np.sqrt(rej_both * (1 - rej_both) / n) + 1e-9
    # a sampler that ignored rejection would fail: the first drafts alone follow q1, not p
    x1 = vector_cascade(1234, p, q1, q2t, 100000)[2]
    assert stats.chisquare(np.bincount(x1, minlength=V), q1 * 100000).pvalue > 1e-3
    assert stats.chisquare(np.bincount(x1, minlength=V), p * 100000).pvalue < 1e-6


class _FakeModel:
    class s:
        R = 4
        n_recurrent = 0
        n_kv_heads = 1
        head_dim = 2


def test_scalar_verify_path_agrees_with_vectorised_composition():
    """Decoder._verify / _draw (the code the scheduler runs) give the same tokens as the vector form."""
    rng = np.random.default_rng(3)
    V, n, T, seed = 12, 3000, 0.8, 99
    z_p, z_1, z_2 = rng.standard_normal(V) * 2, rng.standard_normal(V) * 2, rng.standard_normal(V) * 2
    dec = Decoder(_FakeModel(), temperature=T, seed=seed)
    p, q1, q2t = dec.probs(z_p), dec.probs(z_1), dec.probs(z_2)
    out, src, x1v, x2v, openv = vector_cascade(seed, p, q1, q2t, n)
    for pos in range(n):
        b = Branch(parent=None, token=0, pos=pos - 1, H=None)
        x1, _ = dec._draw(q1, pos, sp.DRAFT1)
        b.records.append(Record(x1, q1, "c1"))
        if q2t[x1] < q1[x1]:
            q2 = sp.residual(q2t, q1)
            x2, _ = dec._draw(q2, pos, sp.DRAFT2)
            b.records.append(Record(x2, q2, "c2"))
            assert x2 == x2v[pos]
        assert x1 == x1v[pos] and (len(b.records) == 2) == bool(openv[pos])
        tok, child, source = dec._verify(b, z_p)
        assert (tok, source) == (out[pos], src[pos])
        assert child == {1: "c1", 2: "c2", 3: None}[source]


def test_race_is_an_exact_categorical_sampler():
    w = np.array([0.0, 3.0, 1.0, 0.0, 6.0])          # unnormalised, with zero-weight entries
    n = 400000
    idx, margin = sp.race(np.broadcast_to(w, (n, 5)), sp.gumbel(5, 3, np.arange(n), sp.VANILLA, 5))
    counts = np.bincount(idx, minlength=5)
    assert counts[0] == 0 and counts[3] == 0
    assert stats.chisquare(counts[[1, 2, 4]], n * w[[1, 2, 4]] / w.sum()).pvalue > 1e-3
    assert (margin >= 0).all()


def test_greedy_verify_reduction():
    """End of Sec. 4.3: first candidate if it is argmax p_R, else the second if present and equal, else argmax."""
    dec = Decoder(_FakeModel(), temperature=0.0)
    z = np.array([0.1, 2.0, 0.3, 1.9])
    for recs, want in [([1], (1, "c1", 1)), ([0], (1, None, 3)), ([0, 1], (1, "c2", 2)), ([0, 3], (1, None, 3))]:
        b = Branch(parent=None, token=0, pos=4, H=None)
        b.records = [Record(t, None, f"c{j + 1}") for j, t in enumerate(recs)]
        assert dec._verify(b, z) == want


# ---- top-k / top-p filters of C (Sec. 3.1) -------------------------------------------------------
def _filter_by_library_sort(p, top_k, top_p):
    """The same filters written with torch's sort and cumsum (nucleus rule as it is usually stated:
    drop a token when the mass ranked strictly before it already reaches top_p)."""
    import torch
    t = torch.tensor(p, dtype=torch.float64)
    V = len(p)
    idx = torch.arange(V)
    # stable sort by decreasing probability keeps lower indices first among equals
    order = torch.sort(-t, stable=True).indices
    keep = torch.ones(V, dtype=torch.bool)
    if top_k and top_k < V:
        keep[order[top_k:]] = False
    t = torch.where(keep, t, torch.zeros_like(t))
    t = t / t.sum()
    if top_p < 1.0:
        ts = t[order]
        before = torch.cumsum(ts, 0) - ts
        drop = before >= top_p
        t[order[drop]] = 0.0
        t = t / t.sum()
    return t.numpy()


@pytest.mark.parametrize("top_k,top_p", [(0, 0.7), (5, 1.0), (6, 0.5), (0, 0.05), (1, 1.0), (3, 0.999)])
def test_filters_match_the_library_sort_formulation_and_are_minimal(top_k, top_p):
    rng = np.random.default_rng(3)
    for V in (2, 7, 16, 300):
        for _ in range(20):
            p = random_dist(rng, V, conc=rng.choice([0.2, 1.0, 5.0]))
            f, margin = sp.top_k_top_p(p, top_k, top_p)
            np.testing.assert_allclose(f, _filter_by_library_sort(p, top_k, top_p), atol=1e-15)
            assert abs(f.sum() - 1) < 1e-12 and margin >= 0
            kept = np.flatnonzero(f)
            # the kept tokens are the most probable ones and stay in proportion
            assert p[kept].min() >= np.delete(p, kept).max(initial=0.0)
            np.testing.assert_allclose(f[kept] / f[kept].sum(), p[kept] / p[kept].sum(), atol=1e-14)
            if top_k:
                assert len(kept) <= top_k
            if top_p < 1.0:      # minimal: dropping the least probable kept token falls short of top_p
                base = np.sort(p)[::-1][: (top_k or V)]
                base = base / base.sum()
                assert base[: len(kept)].sum() >= top_p - 1e-12
                assert len(kept) == 1 or base[: len(kept) - 1].sum() < top_p


def test_filter_special_cases():
    p = np.array([0.1, 0.4, 0.4, 0.1])
    np.testing.assert_allclose(sp.top_k_top_p(p, 0, 1.0)[0], p)                 # both off: C is the plain softmax
    np.testing.assert_allclose(sp.top_k_top_p(p, 1, 1.0)[0], [0, 1, 0, 0])      # ties go to the lower index
    np.testing.assert_allclose(sp.top_k_top_p(p, 0, 0.5)[0], [0, 0.5, 0.5, 0])  # 0.4 < 0.5 <= 0.8
    np.testing.assert_allclose(sp.top_k_top_p(p, 0, 0.4)[0], [0, 1, 0, 0])      # mass 0.4 reaches 0.4
    np.testing.assert_allclose(sp.top_k_top_p(p, 3, 0.9)[0], [1 / 9, 4 / 9, 4 / 9, 0])


@pytest.mark.parametrize("V", [4, 6])
def test_cascade_is_lossless_for_filtered_distributions(V):
    """Losslessness holds for whatever C outputs (Sec. 3.2): with filtered p, q1, q2~ (supports differ, zeros
    inside) the enumerated output law is still the filtered target."""
    rng = np.random.default_rng(11)
    for _ in range(60):
        p, q1, q2t = (sp.top_k_top_p(random_dist(rng, V), int(rng.integers(0, V)), float(rng.uniform(0.3, 1.0)))[0]
                      for _ in range(3))
        law, _, _ = cascade_law(p, q1, q2t)
        np.testing.assert_allclose(law, p, atol=1e-12)
