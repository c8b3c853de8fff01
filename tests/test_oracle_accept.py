"""Pins for the oracle's acceptance rule, residual resample, bonus draw and sampling transform.

The paper prints no numeric example of Eq. 5-6, so these pins are what the mathematics fixes:
exact rational enumeration of the output law on tiny vocabularies (it equals the target
distribution q at beta = 0, the claim that follows Eq. 6, and a closed form for beta > 0),
brute-force inverse CDF, special cases and monotonicity in beta.
"""
from fractions import Fraction as Fr
from itertools import product

import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth

N = 64                                   # grid: midpoints (j + 1/2) / N, exact for dyadic laws
GRID = [(j + 0.5) / N for j in range(N)]


def _law_one_position(p, q, q_bonus, beta):
    """Exact law of (k, y) for gamma = 1 by enumerating x_1 ~ p and grids of r_1, u."""
    V = len(p)
    law = {}
    for x in range(V):
        if p[x] == 0:
            continue
        for r in GRID:
            # the draw used is u_1 on rejection, u_2 on acceptance; enumerate one grid for it
            for u in GRID:
                uni = np.array([[r, u], [0.0, u]])
                res = orc.accept_step(np.array([q, q_bonus], float), np.array([p], float),
                                      np.array([x]), uni, beta)
                key = (res["k"], res["y"])
                law[key] = law.get(key, Fr(0)) + Fr(p[x]).limit_denominator(1 << 20) / (N * N)
    return law


def test_beta_zero_output_law_equals_target_exactly():
    p = [4 / 8, 2 / 8, 1 / 8, 1 / 8]
    q = [1 / 8, 1 / 8, 2 / 8, 4 / 8]
    qb = [2 / 8, 2 / 8, 2 / 8, 2 / 8]
    law = _law_one_position(p, q, qb, 0.0)
    # accepted mass per draft token is p(x) * min(1, q/p) = min(p, q); recover it from the law
    acc_total = sum(v for (k, _), v in law.items() if k == 1)
    assert acc_total == sum(Fr(min(a, b)).limit_denominator(64) for a, b in zip(p, q))
    rej = {y: v for (k, y), v in law.items() if k == 0}
    # residual law: max(0, q - p) / sum  = [0, 0, 1/4, 3/4]; rejected mass = 1 - sum(min(p,q))
    rej_mass = 1 - acc_total
    assert rej == {2: rej_mass * Fr(1, 4), 3: rej_mass * Fr(3, 4)}
    # overall first-token law: min(p,q)(x) + rej_mass * resid(x) == q(x), exactly
    for x in range(4):
        out = Fr(min(p[x], q[x])).limit_denominator(64) + rej.get(x, Fr(0))
        assert out == Fr(q[x]).limit_denominator(64)
    # bonus token after an acceptance follows q_{gamma+1} exactly
    bonus = [sum(v for (k, y), v in law.items() if k == 1 and y == t) for t in range(4)]
    assert bonus == [acc_total * Fr(1, 4)] * 4


@pytest.mark.parametrize("beta", [0.25, 0.5])
def test_beta_positive_output_law_matches_closed_form(beta):
    p = [4 / 8, 2 / 8, 1 / 8, 1 / 8]
    q = [1 / 8, 1 / 8, 2 / 8, 4 / 8]
    qb = [1 / 8, 3 / 8, 2 / 8, 2 / 8]
    law = _law_one_position(p, q, qb, beta)
    A = [min(1.0, min(1.0, q[x] / p[x]) + beta) for x in range(4)]      # P(accept | x)
    acc = sum(Fr(p[x] * A[x]).limit_denominator(1 << 12) for x in range(4))
    assert sum(v for (k, _), v in law.items() if k == 1) == acc
    w = [max(0.0, q[x] - p[x]) for x in range(4)]
    for y in range(4):
        want = (1 - acc) * Fr(w[y] / sum(w)).limit_denominator(64)
        assert law.get((0, y), Fr(0)) == want


def test_two_positions_sequence_law_is_target_ar_law():
    """gamma = 2 with position-dependent targets: emitted tokens follow the target's chain."""
    V = 2
    p1, q1 = [1 / 2, 1 / 2], [1 / 4, 3 / 4]          # ratios 1/2 and 1: exact on the grid
    p2 = {0: [1 / 2, 1 / 2], 1: [1 / 2, 1 / 2]}          # draft row 2 given x_1
    q2 = {0: [1 / 4, 3 / 4], 1: [3 / 4, 1 / 4]}          # target row 2 given x_1
    q3 = [1 / 2, 1 / 2]
    n = 16
    grid = [(j + 0.5) / n for j in range(n)]
    seq_law = {}
    for x1, x2 in product(range(V), range(V)):
        w_draft = Fr(p1[x1]).limit_denominator(8) * Fr(p2[x1][x2]).limit_denominator(8)
        for r1, r2, u in product(grid, grid, grid):
            uni = np.array([[r1, u], [r2, u], [0.0, u]])
            res = orc.accept_step(np.array([q1, q2[x1], q3]), np.array([p1, p2[x1]]),
                                  np.array([x1, x2]), uni, 0.0)
            emitted = tuple([x1, x2][:res["k"]]) + (res["y"],)
            seq_law[emitted] = seq_law.get(emitted, Fr(0)) + w_draft / n ** 3
    assert sum(seq_law.values()) == 1
    first = [sum(v for s, v in seq_law.items() if s[0] == t) for t in range(V)]
    assert first == [Fr(1, 4), Fr(3, 4)]                              # = q1
    # given x_1 = a was accepted (sequence has >= 2 tokens), the second token follows q2[a]
    for a in range(V):
        mass = sum(v for s, v in seq_law.items() if len(s) >= 2 and s[0] == a)
        for b in range(V):
            got = sum(v for s, v in seq_law.items() if len(s) >= 2 and s[:2] == (a, b))
            assert got == mass * Fr(q2[a][b]).limit_denominator(8)
    # three tokens only when both drafts were accepted; the third follows q3
    m3 = sum(v for s, v in seq_law.items() if len(s) == 3)
    assert sum(v for s, v in seq_law.items() if len(s) == 3 and s[2] == 0) == m3 * Fr(1, 2)


def test_control_flow_properties_random():
    rng = np.random.default_rng(0)
    V, gamma = 11, 4
    for trial in range(300):
        q = rng.dirichlet(np.ones(V), size=gamma + 1)
        p = rng.dirichlet(np.ones(V), size=gamma)
        x = np.array([rng.choice(V, p=p[i]) for i in range(gamma)])
        uni = rng.random((gamma + 1, 2))
        prev_k = -1
        for beta in [0.0, 0.1, 0.4, 1.0]:
            res = orc.accept_step(q, p, x, uni, beta)
            k, y = res["k"], res["y"]
            assert 0 <= k <= gamma and 0 <= y < V
            assert k >= prev_k                       # larger beta never accepts fewer
            prev_k = k
            th = res["thresholds"]
            assert all(uni[i, 0] < th[i] for i in range(k))
            if k < gamma:
                assert uni[k, 0] >= th[k]
                resid = np.maximum(0, q[k] - p[k])
                assert resid[y] > 0                  # resampled token has residual mass
                assert y != x[k]                     # a rejected token has q < p: no residual
            else:
                assert q[gamma][y] > 0
        assert prev_k == gamma                       # beta >= 1 accepts everything (r < 1)


def test_identical_distributions_always_accept():
    rng = np.random.default_rng(1)
    q = rng.dirichlet(np.ones(7), size=4)
    x = np.array([2, 5, 0])
    res = orc.accept_step(q, q[:3].copy(), x, rng.random((4, 2)) * 0.999999, 0.0)
    assert res["k"] == 3


def test_zero_draft_probability_does_not_divide():
    q = np.array([[0.5, 0.5], [0.5, 0.5]])
    p = np.array([[0.0, 1.0]])
    res = orc.accept_step(q, p, np.array([0]), np.array([[0.99, 0.3], [0.0, 0.3]]), 0.0)
    assert res["k"] == 1 and res["thresholds"][0] == 1.0


def test_zero_residual_falls_back_to_target_row():
    q = np.array([[0.25, 0.75], [0.5, 0.5]])
    p = q[:1].copy()                                  # p == q: residual is identically zero
    # force a "rejection" with r >= 1 (not reachable with r in [0,1), exercised directly)
    res = orc.accept_step(q, p, np.array([1]), np.array([[1.5, 0.1], [0.0, 0.0]]), 0.0)
    assert res["k"] == 0 and res["y"] == 0            # u = 0.1 < 0.25 -> id 0 of q itself


def test_categorical_draw_brute_force():
    rng = np.random.default_rng(2)
    for _ in range(200):
        V = int(rng.integers(1, 9))
        w = rng.random(V) * (rng.random(V) > 0.3)
        if w.sum() == 0:
            w[rng.integers(V)] = 1.0
        u = float(rng.random())
        acc, want = 0.0, None
        for t in range(V):                            # definition: first id whose CDF exceeds u*S
            acc += w[t]
            if acc > u * w.sum():
                want = t
                break
        got, margin = orc.categorical_draw(w, u)
        assert got == want and w[got] > 0 and margin >= 0


def test_categorical_draw_frequencies():
    w = np.array([1.0, 0.0, 3.0, 4.0])
    counts = np.zeros(4)
    n = 8000
    for j in range(n):
        counts[orc.categorical_draw(w, (j + 0.5) / n)[0]] += 1
    assert np.array_equal(counts, [1000, 0, 3000, 4000])


def test_transform_against_torch_and_special_cases():
    rng = np.random.default_rng(3)
    z = rng.standard_normal(50) * 3
    q = orc.transform(z, 0.8, 0)
    ref = torch.softmax(torch.from_numpy(z) / 0.8, dim=0).numpy()
    assert np.allclose(q, ref, atol=1e-15)
    assert np.allclose(orc.transform(z, 0.8, 50), q) and np.allclose(orc.transform(z, 0.8, 500), q)
    qk = orc.transform(z, 0.8, 5)
    top = torch.topk(torch.from_numpy(z), 5)
    assert set(np.nonzero(qk)[0]) == set(top.indices.tolist())
    assert np.isclose(qk.sum(), 1.0)
    ref_k = torch.softmax(top.values / 0.8, dim=0).numpy()
    assert np.allclose(qk[top.indices.numpy()], ref_k, atol=1e-15)
    # ties at the cut: the lower id is kept
    zt = np.array([1.0, 5.0, 5.0, 5.0, 0.0])
    assert list(np.nonzero(orc.transform(zt, 1.0, 2))[0]) == [1, 2]
    # shift invariance and temperature -> argmax
    assert np.allclose(orc.transform(z + 100.0, 1.0, 0), orc.transform(z, 1.0, 0))
    assert orc.transform(z, 1e-3, 0).argmax() == z.argmax()


def test_nucleus_transform_by_hand_brute_force_and_library():
    """top-p keeps the shortest most-probable-first prefix whose mass reaches top_p."""
    # by hand: probabilities 0.5, 0.3, 0.15, 0.05 (ids shuffled)
    pr = np.array([0.15, 0.5, 0.05, 0.3])
    z = np.log(pr)
    assert list(np.nonzero(orc.transform(z, 1.0, 0, 0.79))[0]) == [1, 3]          # 0.5 + 0.3 reaches 0.79
    assert list(np.nonzero(orc.transform(z, 1.0, 0, 0.81))[0]) == [0, 1, 3]       # needs the third
    assert list(np.nonzero(orc.transform(z, 1.0, 0, 0.4))[0]) == [1]
    q = orc.transform(z, 1.0, 0, 0.79)
    assert np.allclose(q[[1, 3]], [0.5 / 0.8, 0.3 / 0.8]) and np.isclose(q.sum(), 1.0)
    assert np.allclose(orc.transform(z, 1.0, 0, 0.0), pr) and np.allclose(orc.transform(z, 1.0, 0, 1.0), pr)
    # ties: equal probabilities enter in id order
    zt = np.log(np.array([0.25, 0.25, 0.25, 0.25]))
    assert list(np.nonzero(orc.transform(zt, 1.0, 0, 0.5))[0]) == [0, 1]
    assert list(np.nonzero(orc.transform(zt, 1.0, 0, 0.51))[0]) == [0, 1, 2]
    # after top-k the nucleus is taken inside the kept set (mass relative to that set)
    assert list(np.nonzero(orc.transform(z, 1.0, 2, 0.7))[0]) == [1, 3]            # 0.5/0.8 = 0.625 < 0.7
    assert list(np.nonzero(orc.transform(z, 1.0, 2, 0.6))[0]) == [1]
    # brute force: among all most-probable-first prefixes, the shortest with mass >= top_p
    rng = np.random.default_rng(11)
    for _ in range(200):
        V = int(rng.integers(2, 9))
        zz = rng.standard_normal(V) * 2
        T = float(rng.uniform(0.5, 1.5))
        top_p = float(rng.uniform(0.05, 0.98))
        full = orc.transform(zz, T, 0)
        order = np.argsort(-full, kind="stable")
        n = next(i + 1 for i in range(V) if full[order[:i + 1]].sum() >= top_p or i == V - 1)
        got = orc.transform(zz, T, 0, top_p)
        assert set(np.nonzero(got)[0]) == set(order[:n].tolist())
        assert np.allclose(got[order[:n]], full[order[:n]] / full[order[:n]].sum())
    # library routine: the nucleus filter of `transformers`
    from transformers.generation.logits_process import TopPLogitsWarper
    for seed in range(20):
        zz = np.random.default_rng(seed).standard_normal(64) * 2.5
        tp = 0.3 + 0.03 * seed
        kept_ref = torch.isfinite(TopPLogitsWarper(top_p=tp)(None, torch.from_numpy(zz)[None].clone()))[0].numpy()
        assert np.array_equal(orc.transform(zz, 1.0, 0, tp) > 0, kept_ref)


def test_repetition_aware_law_by_enumerating_the_two_stage_procedure():
    """The closed form of transform_ras against a literal enumeration of the procedure: first draw
    from the nucleus row; if that id is repeated in the window, second draw from the full row."""
    rng = np.random.default_rng(8)
    for trial in range(60):
        V = int(rng.integers(4, 10))
        z = rng.standard_normal(V) * 2
        T = float(rng.uniform(0.6, 1.4))
        top_k = int(rng.integers(0, V + 1))
        top_p = float(rng.choice([0.0, 0.5, 0.8, 0.95]))
        win = int(rng.integers(1, 8))
        tau = float(rng.choice([0.1, 0.3, 0.5]))
        window = rng.integers(-1, V, size=int(rng.integers(0, 12)))
        q_nuc, q_full = orc.transform(z, T, top_k, top_p), orc.transform(z, T, 0)
        tail = [int(t) for t in window[-win:] if t >= 0]
        law = np.zeros(V)
        for first in range(V):
            if q_nuc[first] == 0:
                continue
            if tail.count(first) >= win * tau:
                law += q_nuc[first] * q_full                 # thrown away, redrawn from the full row
            else:
                law[first] += q_nuc[first]
        got = orc.transform_ras(z, T, top_k, top_p, window, win, tau)
        assert np.allclose(got, law, atol=1e-14) and np.isclose(got.sum(), 1.0)
    z = np.log(np.array([0.5, 0.3, 0.15, 0.05]))
    # by hand: nucleus {0, 1} = (0.625, 0.375); id 0 repeated -> 0.625 of the mass is redrawn from the full row
    got = orc.transform_ras(z, 1.0, 0, 0.79, np.array([3, 0, 2]), 10, 0.1)
    assert np.allclose(got, [0.625 * 0.5, 0.375 + 0.625 * 0.3, 0.625 * 0.15, 0.625 * 0.05])
    # no window, an empty window, or a threshold no count reaches: the nucleus row itself
    nuc = orc.transform(z, 1.0, 0, 0.79)
    assert np.allclose(orc.transform_ras(z, 1.0, 0, 0.79, np.array([0, 0]), 0, 0.1), nuc)
    assert np.allclose(orc.transform_ras(z, 1.0, 0, 0.79, np.array([-1, -1]), 4, 0.1), nuc)
    assert np.allclose(orc.transform_ras(z, 1.0, 0, 0.79, np.array([0, 1]), 4, 0.9), nuc)
    # only the last win_size tokens count
    assert np.allclose(orc.transform_ras(z, 1.0, 0, 0.79, np.array([0, 2, 2, 3]), 3, 0.3), nuc)
    # every kept id repeated: the full row
    assert np.allclose(orc.transform_ras(z, 1.0, 0, 0.79, np.array([0, 1]), 2, 0.5), orc.transform(z, 1.0, 0))


def test_verify_builds_each_rows_window_from_recent_tokens_and_the_draft():
    from tests.helpers import oracle_model, small_shape
    from paper_2505_15380_b200 import synth
    shape = small_shape()
    m = oracle_model(shape, synth.make_weights(shape, 2))
    st = orc.Stream(m, 64)
    orc.prefill(m, st, np.array([5, 9, 3, 9, 7]))
    draft = np.array([9, 9, 4])
    V = shape.vocab_out
    p = np.full((3, V), 1.0 / V)
    u = np.zeros((4, 2))
    recent = np.array([3, 9, 7])
    o = orc.verify(m, st, draft, p, u, temperature=1.0, top_k=5, beta=0.0, top_p=0.9, recent=recent,
                   win_size=4, tau_r=0.5)
    lg = o["logits"]
    for i in range(4):
        window = np.concatenate([recent, draft[:i]])        # row i sees x_1..x_{i-1}, not x_i
        assert np.allclose(o["q_rows"][i], orc.transform_ras(lg[i], 1.0, 5, 0.9, window, 4, 0.5))
    # row 2's window is [9, 7, 9, 9]: id 9 occurs 3 >= 2 times, so its nucleus mass is spread
    assert not np.allclose(o["q_rows"][2], orc.transform(lg[2], 1.0, 5, 0.9)) or orc.transform(lg[2], 1.0, 5, 0.9)[9] == 0


def test_accepted_length_grows_with_beta_as_in_table_3():
    """Sec. 4.3 / Table 3: a larger tolerance accepts more.  For fixed distributions, tokens and
    uniforms k(beta) never decreases, and its mean over draws follows the geometric closed form
    with the per-position acceptance probability A = sum_x p(x) min(1, min(1, q/p) + beta)."""
    rng = np.random.default_rng(5)
    V, gamma, n = 12, 3, 4000
    q = rng.dirichlet(np.ones(V) * 0.7)
    p = rng.dirichlet(np.ones(V) * 0.7)
    qs, ps = np.tile(q, (gamma + 1, 1)), np.tile(p, (gamma, 1))
    means = []
    for beta in (0.0, 0.1, 0.2, 0.3, 0.4):
        ks = []
        for i in range(n):
            r = np.random.default_rng(1000 + i)
            x = r.choice(V, size=gamma, p=p)
            u = r.random((gamma + 1, 2))
            ks.append(orc.accept_step(qs, ps, x, u, beta)["k"])
        means.append(np.mean(ks))
        A = float(np.sum(p * np.minimum(1.0, np.minimum(1.0, q / p) + beta)))
        closed = sum(A ** j for j in range(1, gamma + 1))          # E[k] = A + A^2 + ... + A^gamma
        assert abs(means[-1] - closed) < 4 * np.sqrt(gamma / n) + 0.02
    assert all(b >= a for a, b in zip(means, means[1:])) and means[-1] > means[0] + 0.3
    # same draws, larger beta: never fewer accepted
    for i in range(200):
        r = np.random.default_rng(i)
        x = r.choice(V, size=gamma, p=p)
        u = r.random((gamma + 1, 2))
        kk = [orc.accept_step(qs, ps, x, u, b)["k"] for b in (0.0, 0.1, 0.2, 0.3, 0.4, 1.0)]
        assert kk == sorted(kk) and kk[-1] == gamma


def test_expected_tokens_per_iteration_geometric_identity():
    """With i.i.d. acceptance probability alpha, E[k+1] = (1 - alpha^(gamma+1)) / (1 - alpha)."""
    V, gamma, alpha = 4, 4, 0.5
    p = np.tile(np.array([0.5, 0.5, 0.0, 0.0]), (gamma, 1))
    q = np.tile(np.array([0.25, 0.25, 0.25, 0.25]), (gamma + 1, 1))      # q/p = 1/2 on support
    uni = synth.verify_uniforms(7, 4000, gamma + 1).astype(np.float64)
    tot = 0
    for b in range(4000):
        tot += orc.accept_step(q, p, np.zeros(gamma, int), uni[b], 0.0)["k"] + 1
    want = (1 - alpha ** (gamma + 1)) / (1 - alpha)
    assert abs(tot / 4000 - want) < 0.06


def test_verify_wires_rows_to_positions():
    """Row i of the forward is tested against draft token i+1 (a shifted index must fail)."""
    from tests.helpers import oracle_model, small_shape
    shape = small_shape()
    w = synth.make_weights(shape, 4)
    m = oracle_model(shape, w)
    st = orc.Stream(m, 32)
    orc.prefill(m, st, np.arange(9) % shape.vocab_in)
    draft = np.array([3, 7, 11])
    logits = orc.forward(m, st, np.concatenate([[st.pending], draft]))
    q_rows = np.stack([orc.transform(r, 1.0, 0) for r in logits])
    p_rows = q_rows[:3].copy().astype(np.float32)                 # p == q: must accept all
    res = orc.verify(m, st, draft, p_rows, np.full((4, 2), 0.999), temperature=1.0, top_k=0,
                     beta=0.0)
    assert res["k"] == 3
    p_bad = np.roll(q_rows[:3], 1, axis=0).astype(np.float32)     # mis-indexed rows
    p_bad[:, draft] *= 50.0
    res2 = orc.verify(m, st, draft, p_bad, np.full((4, 2), 0.999), temperature=1.0, top_k=0,
                      beta=0.0)
    assert res2["k"] < 3
    assert np.allclose(res["logits"], logits)
