"""Pins of the CPU oracle against things other than itself (Sec. 3.1 Eq. 2-4, Sec. 3.3 Eq. 5-10).

Library routines (scipy softmax, numpy matmul), closed forms, hand-worked fixtures, brute force on
tiny inputs and structural invariants; chosen so that a dropped term, a wrong sign/index or a
transposed operand in the oracle fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import lar_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ decode attention (Eq. 2-3)
@pytest.mark.parametrize("n,d", [(1, 8), (7, 16), (33, 64), (150, 128), (5, 3)])
def test_attention_matches_library_softmax_matmul(n, d):
    q, K, V = rng.normal(size=d), rng.normal(size=(n, d)), rng.normal(size=(n, d))
    scale = 1.0 / math.sqrt(d)
    out, p = O.attention(q, K, V, scale, want_probs=True)
    ref_p = sp_softmax((K @ q) * scale)
    np.testing.assert_allclose(p, ref_p, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(out, ref_p @ V, rtol=1e-12, atol=1e-14)
    assert abs(p.sum() - 1.0) < 1e-6


def test_attention_two_key_closed_form_pins_the_scale():
    # two keys: p_1 = sigmoid((q.k1 - q.k2) / sqrt(d)); a dropped or squared sqrt(d) fails
    d = 16
    q = np.zeros(d); q[0] = 2.0
    K = np.zeros((2, d)); K[0, 0] = 3.0; K[1, 0] = 1.0
    V = np.array([[1.0] * d, [0.0] * d])
    out = O.attention(q, K, V, 1.0 / math.sqrt(d))
    expect = 1.0 / (1.0 + math.exp(-(6.0 - 2.0) / 4.0))
    np.testing.assert_allclose(out, expect, rtol=1e-14)


def test_attention_invariants():
    n, d = 40, 32
    q, K, V = rng.normal(size=d), rng.normal(size=(n, d)), rng.normal(size=(n, d))
    s = 1 / math.sqrt(d)
    out = O.attention(q, K, V, s)
    # convex combination: inside the per-dimension range of V
    assert np.all(out <= V.max(0) + 1e-12) and np.all(out >= V.min(0) - 1e-12)
    # constant V -> constant output
    np.testing.assert_allclose(O.attention(q, K, np.full((n, d), 2.5), s), 2.5, rtol=1e-14)
    # invariant to a permutation of the cache slots
    perm = rng.permutation(n)
    np.testing.assert_allclose(O.attention(q, K[perm], V[perm], s), out, rtol=1e-12, atol=1e-14)
    # logit shift invariance: adding a vector orthogonal to nothing but constant across keys
    # (q.(k + c) = q.k + q.c for all keys) leaves the softmax unchanged
    c = rng.normal(size=d)
    np.testing.assert_allclose(O.attention(q, K + c, V, s), out, rtol=1e-10, atol=1e-12)
    # large logits do not overflow (max subtraction)
    big = O.attention(q * 1e3, K, V, s)
    assert np.all(np.isfinite(big))
    j = int(np.argmax(K @ q))
    np.testing.assert_allclose(big, V[j], atol=1e-9)


# ------------------------------------------------------------------ saliency (Eq. 9)
def _golden_2x3():
    vals = {}
    for line in open(os.path.join(GOLD, "saliency_2x3.txt")):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":")
        vals[k.strip()] = [int(x) for x in v.split()]
    return vals


def test_saliency_hand_worked_fixture():
    g = _golden_2x3()
    a = np.array(g["a"], dtype=float)
    Kmid = np.stack([math.sqrt(2.0) * np.log(a), np.zeros(3)], axis=1)
    Qg = np.array([[1.0, 0.0], [-1.0, 0.0]])
    S = O.saliency(Qg, Kmid, 1.0 / math.sqrt(2.0))
    np.testing.assert_allclose(S, np.array(g["S_num"]) / g["S_den"][0], rtol=1e-13)
    pos = np.arange(3) + 10
    assert list(O.bottomk(S, pos, 1)) == g["bottom1"]
    assert list(O.bottomk(S, pos, 2)) == g["bottom2"]


@pytest.mark.parametrize("nq,M,d", [(1, 5, 4), (24, 48, 128), (49, 147, 64), (7, 3, 5)])
def test_saliency_matches_library_and_sums_to_one(nq, M, d):
    Qg, Km = rng.normal(size=(nq, d)), rng.normal(size=(M, d))
    scale = 1 / math.sqrt(d)
    S = O.saliency(Qg, Km, scale)
    ref = sp_softmax((Qg @ Km.T) * scale, axis=1).mean(axis=0)
    np.testing.assert_allclose(S, ref, rtol=1e-12, atol=1e-16)
    # every query contributes total mass exactly 1 -> the scores sum to 1
    assert abs(S.sum() - 1.0) < 1e-12


def test_saliency_is_mean_over_queries_and_heads():
    # scoring with all rows == mean of scoring with each row alone (equal contribution, Eq. 9)
    nq, M, d = 6, 9, 8
    Qg, Km = rng.normal(size=(nq, d)), rng.normal(size=(M, d))
    s = 0.3
    whole = O.saliency(Qg, Km, s)
    parts = np.mean([O.saliency(Qg[j:j + 1], Km, s) for j in range(nq)], axis=0)
    np.testing.assert_allclose(whole, parts, rtol=1e-13)
    # one dominant key collects (almost) all the mass
    Km2 = Km.copy(); Km2[4] = 0
    Qpos = np.abs(rng.normal(size=(nq, d)))
    Km2[4] = 50.0
    S = O.saliency(Qpos, Km2, s)
    assert S[4] > 1 - 1e-9
    # uniform keys -> uniform scores
    S = O.saliency(Qg, np.tile(Km[:1], (M, 1)), s)
    np.testing.assert_allclose(S, 1.0 / M, rtol=1e-13)


# ------------------------------------------------------------------ BottomK (Eq. 10)
def _brute_bottomk(S, pos, k):
    order = sorted(range(len(S)), key=lambda m: (S[m], -pos[m]))
    return order[:k]


@pytest.mark.parametrize("M,k", [(1, 1), (5, 2), (16, 16), (48, 16), (31, 7)])
def test_bottomk_vs_brute_force_sort_with_ties(M, k):
    for trial in range(20):
        S = rng.integers(0, 4, size=M).astype(float) / 4.0 if trial % 2 == 0 else rng.random(M)
        pos = np.sort(rng.choice(1000, size=M, replace=False)).astype(np.int32)
        assert list(O.bottomk(S, pos, k)) == _brute_bottomk(S, pos, k)


def test_bottomk_tie_break_evicts_newest():
    S = np.full(6, 0.25)
    pos = np.array([3, 5, 9, 11, 20, 21], dtype=np.int32)
    assert list(O.bottomk(S, pos, 2)) == [5, 4]


# ------------------------------------------------------------------ pipeline (Eq. 5-8)
def _run_unit(cfg, inputs, record=None):
    u = O.Unit(cfg)
    C, n, N = cfg.cond_len, cfg.line_width, cfg.line_width * cfg.n_lines
    u.prefill(inputs["kc"], inputs["vc"])
    outs, lens, events = [], [], []
    for i in range(N):
        outs.append(u.step(inputs["q"][i], inputs["k"][i], inputs["v"][i]))
        lens.append(u.len)
        if (i + 1) % n == 0 and (i + 1) < N:
            ev = u.line_end()
            events.append((i + 1, ev, u.positions().copy()))
    return np.array(outs), lens, events, u


def _rand_inputs(C, N, G, d, seed=0):
    r = np.random.default_rng(seed)
    f = lambda *s: r.normal(size=s).astype(np.float32)
    return {"q": f(N, G, d), "k": f(N, d), "v": f(N, d), "kc": f(C, d), "vc": f(C, d)}


def test_budget_at_least_sequence_length_equals_full_attention_exactly():
    C, n, h, G, d = 3, 4, 5, 2, 8
    inp = _rand_inputs(C, n * h, G, d)
    full, _, _, _ = _run_unit(O.make_cfg(C, n, h, h, 2, 1, G, d), inp)
    big, _, ev, _ = _run_unit(O.make_cfg(C, n, h, h + 3, 2, 1, G, d), inp)
    assert np.array_equal(full, big) and all(e[1] is None for e in ev)
    # and the full path is Eq. 2 over [K_cond, K_1:i] (library check at every step)
    s = 1 / math.sqrt(d)
    for i in range(n * h):
        K = np.concatenate([inp["kc"], inp["k"][: i + 1]]).astype(np.float64)
        V = np.concatenate([inp["vc"], inp["v"][: i + 1]]).astype(np.float64)
        for g in range(G):
            ref = sp_softmax((K @ inp["q"][i, g].astype(np.float64)) * s) @ V
            np.testing.assert_allclose(full[i, g], ref, rtol=1e-12, atol=1e-14)


def test_toy_8x8_ratio_three_eighths_trajectory():
    # Fig. 2's toy case: 8x8 grid, rho = 3/8 -> B = 24; no compression before the end of line 3,
    # then every line end leaves B - n = 16 visual entries; 5 compressions (lines 3..7).
    C, n, h, G, d = 2, 8, 8, 1, 4
    cfg = O.make_cfg(C, n, h, 3, 4, 1, G, d)
    inp = _rand_inputs(C, n * h, G, d, seed=3)
    _, lens, events, _ = _run_unit(cfg, inp)
    B = 24
    for i, L in enumerate(lens, start=1):
        expect = i if i <= B else B - n + ((i - 1) % n + 1)
        assert L - C == expect
        assert L - C <= B
    compress = [(i, ev) for i, ev, _ in events if ev is not None]
    assert [i // n for i, _ in compress] == [3, 4, 5, 6, 7]
    for i, ev, pos in events:
        if ev is not None:
            assert len(pos) - C == B - n


def test_retention_invariant_and_evictions_only_from_mid():
    C, n, h, G, d = 5, 6, 10, 2, 16
    N_init, r, bl = 4, 2, 5
    cfg = O.make_cfg(C, n, h, bl, N_init, r, G, d)
    inp = _rand_inputs(C, n * h, G, d, seed=7)
    _, _, events, _ = _run_unit(cfg, inp)
    prev = None
    for i, ev, pos in events:
        l = i // n
        pos = list(pos)
        assert pos == sorted(pos) and len(set(pos)) == len(pos)
        assert pos[:C] == list(range(C))                                   # prefix always kept
        if ev is None:
            assert len(pos) == C + i
            continue
        vis = [p - C + 1 for p in pos[C:]]
        assert set(range(1, N_init + 1)) <= set(vis)                        # anchor kept
        assert set(range((l - r) * n + 1, l * n + 1)) <= set(vis)           # last r lines kept
        assert len(ev["evicted_pos"]) == n and len(set(ev["evicted_pos"])) == n
        for p in ev["evicted_pos"]:
            vi = p - C + 1
            assert N_init < vi <= (l - r) * n and p in set(ev["mid_pos"])
        M = bl * n - N_init - r * n
        assert len(ev["mid_pos"]) == M
        # the evicted ones are exactly the n lowest under (score asc, position desc)
        order = sorted(range(M), key=lambda m: (ev["scores"][m], -ev["mid_pos"][m]))
        assert sorted(ev["mid_pos"][order[:n]]) == sorted(ev["evicted_pos"])
        assert ev["boundary"][0] >= ev["boundary"][1]
        assert abs(ev["scores"].sum() - 1) < 1e-12


def test_mid_equals_one_line_gives_closed_form_init_plus_recent():
    # M = n: the whole mid region goes at every line end, whatever the scores
    C, n, h, G, d = 2, 4, 9, 1, 8
    N_init, r = 4, 2
    bl = (N_init + r * n + n) // n
    cfg = O.make_cfg(C, n, h, bl, N_init, r, G, d)
    _, _, events, _ = _run_unit(cfg, _rand_inputs(C, n * h, G, d, seed=11))
    for i, ev, pos in events:
        if ev is None:
            continue
        l = i // n
        expect = list(range(C)) + [C + v - 1 for v in range(1, N_init + 1)] + \
                 [C + v - 1 for v in range((l - r) * n + 1, l * n + 1)]
        assert list(pos) == expect


def test_uniform_mid_keys_evict_the_newest_mid_tokens():
    C, n, h, G, d = 1, 4, 8, 1, 8
    N_init, r, bl = 4, 1, 4
    inp = _rand_inputs(C, n * h, G, d, seed=5)
    inp["k"][:] = inp["k"][0]                       # all visual keys equal -> uniform scores
    cfg = O.make_cfg(C, n, h, bl, N_init, r, G, d)
    _, _, events, _ = _run_unit(cfg, inp)
    for i, ev, pos in events:
        if ev is None:
            continue
        np.testing.assert_allclose(ev["scores"], 1.0 / len(ev["scores"]), rtol=1e-12)
        assert sorted(ev["evicted_pos"]) == sorted(ev["mid_pos"])[-n:]


def test_scores_use_current_line_queries_and_mid_keys_only():
    # Re-derive one line end from the raw inputs with library routines: the guide queue must hold
    # exactly the queries of the finished line, the keys exactly the mid region (Eq. 8-9).
    C, n, h, G, d = 3, 5, 6, 2, 8
    N_init, r, bl = 2, 1, 3
    cfg = O.make_cfg(C, n, h, bl, N_init, r, G, d)
    inp = _rand_inputs(C, n * h, G, d, seed=21)
    _, _, events, _ = _run_unit(cfg, inp)
    i, ev, pos = next(e for e in events if e[1] is not None)
    l = i // n
    assert l == bl
    mid_vis = [v for v in range(N_init + 1, (l - r) * n + 1)]
    assert list(ev["mid_pos"]) == [C + v - 1 for v in mid_vis]
    Qg = inp["q"][(l - 1) * n: l * n].reshape(n * G, d).astype(np.float64)
    Km = inp["k"][[v - 1 for v in mid_vis]].astype(np.float64)
    ref = sp_softmax(Qg @ Km.T / math.sqrt(d), axis=1).mean(0)
    np.testing.assert_allclose(ev["scores"], ref, rtol=1e-12)


def test_compressed_output_is_attention_over_the_kept_set():
    # after compressions, a step's output equals library attention over exactly the kept entries
    C, n, h, G, d = 2, 4, 7, 1, 8
    cfg = O.make_cfg(C, n, h, 3, 2, 1, G, d)
    inp = _rand_inputs(C, n * h, G, d, seed=33)
    u = O.Unit(cfg)
    u.prefill(inp["kc"], inp["vc"])
    allK = np.concatenate([inp["kc"], inp["k"]]).astype(np.float64)
    allV = np.concatenate([inp["vc"], inp["v"]]).astype(np.float64)
    for i in range(n * h):
        out, probs = u.step(inp["q"][i], inp["k"][i], inp["v"][i], want_probs=True)
        pos = u.positions()
        ref = sp_softmax(allK[pos] @ inp["q"][i, 0].astype(np.float64) / math.sqrt(d)) @ allV[pos]
        np.testing.assert_allclose(out[0], ref, rtol=1e-12, atol=1e-14)
        assert abs(probs.sum() - 1.0) < 1e-6
        if (i + 1) % n == 0 and i + 1 < n * h:
            u.line_end()


def test_call_order_errors():
    cfg = O.make_cfg(1, 2, 3, 2, 0, 0, 1, 4)   # r = 0 allowed by the oracle, B=4, M=4
    inp = _rand_inputs(1, 6, 1, 4)
    u = O.Unit(cfg)
    u.prefill(inp["kc"], inp["vc"])
    u.step(inp["q"][0], inp["k"][0], inp["v"][0])
    assert u.line_end_due() == -1
    u.step(inp["q"][1], inp["k"][1], inp["v"][1])
    with pytest.raises(RuntimeError):
        u.step(inp["q"][2], inp["k"][2], inp["v"][2])   # line complete: line end is due first
    with pytest.raises(ValueError):
        O.Unit(O.make_cfg(1, 4, 8, 2, 4, 1, 1, 4))       # B - N_init - r n = 0 < n


def test_run_units_matches_stepwise_driver():
    from paper_2512_04857_b200 import workloads as W
    w = W.WORKLOADS["tiny_b"]
    cfg = O.cfg_from_workload(w)
    units = [W.gen_unit(w, 0, 0, hk) for hk in (0, 5)]
    st = lambda key: np.stack([u[key].numpy() for u in units])
    out, kept, thr = O.run_units(cfg, st("q"), st("k"), st("v"), st("kc"), st("vc"))
    assert thr >= 1
    for ui, unit in enumerate(units):
        o2, _, events, _ = _run_unit(cfg, {k: v.numpy() for k, v in unit.items()})
        assert np.array_equal(out[ui], o2)
        for li, (_, ev, pos) in enumerate(events):
            row = kept[ui, li]
            assert list(row[row >= 0]) == list(pos)


# ------------------------------------------------- variant of Eq. 9: normalised over the whole live cache
def _drive_one_line(cfg, seed, want_probs):
    """Prefill, run to the first compressing line end; returns the unit and the last line's step probabilities."""
    r = np.random.default_rng(seed)
    C_, n, G, d = cfg.cond_len, cfg.line_width, cfg.group, cfg.head_dim
    u = O.Unit(cfg)
    u.prefill(r.normal(size=(C_, d)), r.normal(size=(C_, d)))
    probs = []
    for i in range(cfg.budget_lines * n):
        res = u.step(r.normal(size=(G, d)), r.normal(size=d), r.normal(size=d), want_probs=want_probs)
        if want_probs and i >= (cfg.budget_lines - 1) * n:
            probs.append(res[1])
        if (i + 1) % n == 0 and (i + 1) < cfg.budget_lines * n:
            assert u.line_end() is None
    assert u.line_end_due() == 1
    return u, probs


@pytest.mark.parametrize("G", [1, 3])
def test_cache_normalised_scores_are_the_decode_probabilities_of_the_line(G):
    # the variant's score of a mid token = mean over the line's steps and heads of the probability Eq. 2-3 gave it
    # at that step (those probabilities are pinned to the library softmax above)
    cfg = O.make_cfg(5, 6, 10, 5, 4, 2, G, 16, score_norm=1)
    u, probs = _drive_one_line(cfg, 77, True)
    S, mid_pos = u.mid_scores()
    pos = u.positions()
    slot_of = {int(p): s for s, p in enumerate(pos)}
    expect = np.zeros(len(mid_pos))
    for p_t in probs:                       # [G][len at that step]; slots do not move within a line
        for m, mp in enumerate(mid_pos):
            expect[m] += p_t[:, slot_of[int(mp)]].sum()
    expect /= cfg.line_width * G
    np.testing.assert_allclose(S, expect, rtol=1e-12, atol=1e-15)
    assert 0.0 < S.sum() < 1.0              # the mid region holds only part of every query's mass


def test_cache_normalised_scores_vs_library_softmax_with_causal_cut():
    r = np.random.default_rng(5)
    n, G, d, ln = 4, 2, 8, 19
    Qg, K = r.normal(size=(n, G, d)), r.normal(size=(ln, d))
    pos = np.arange(ln) + 3                 # any increasing positions
    first_qpos = int(pos[ln - n])
    mid = [2, 3, 5, 6, 7, 9]
    S = O.saliency_cache(Qg, K, pos, first_qpos, mid, 0.3)
    expect = np.zeros(len(mid))
    for t in range(n):
        live = ln - n + t + 1               # entries appended up to and including query t's own token
        for g in range(G):
            expect += sp_softmax((K[:live] @ Qg[t, g]) * 0.3)[mid]
    np.testing.assert_allclose(S, expect / (n * G), rtol=1e-12, atol=1e-15)


def test_cache_normalisation_reduces_to_eq9_when_only_the_mid_keys_carry_mass():
    # every key outside the mid region points away from all queries with a huge norm: its probability underflows
    # to zero and the two readings of Eq. 9 coincide
    r = np.random.default_rng(9)
    n, G, d, ln = 3, 2, 6, 14
    Qg = np.abs(r.normal(size=(n, G, d)))
    K = r.normal(size=(ln, d))
    mid = [4, 5, 6, 7, 8]
    for s in range(ln):
        if s not in mid:
            K[s] = -1e3
    pos = np.arange(ln)
    a = O.saliency_cache(Qg, K, pos, ln - n, mid, 1.0)
    b = O.saliency(Qg.reshape(n * G, d), K[mid], 1.0)
    np.testing.assert_allclose(a, b, rtol=1e-12)
    assert abs(a.sum() - 1.0) < 1e-9


def test_the_two_normalisations_differ_and_can_change_the_kept_set():
    cfg0 = O.make_cfg(5, 6, 10, 5, 4, 2, 2, 16, score_norm=0)
    cfg1 = O.make_cfg(5, 6, 10, 5, 4, 2, 2, 16, score_norm=1)
    u0, _ = _drive_one_line(cfg0, 3, False)
    u1, _ = _drive_one_line(cfg1, 3, False)
    S0, p0 = u0.mid_scores()
    S1, p1 = u1.mid_scores()
    assert (p0 == p1).all()
    assert abs(S0.sum() - 1.0) < 1e-9 and S1.sum() < 0.9
    assert not np.allclose(S0 / S0.sum(), S1 / S1.sum(), rtol=1e-3)


# ------------------------------------------------- accumulated attention over all history (the "w. AttAcc" ablation)
def _drive_generation(cfg, seed, on_step=None, on_line_end=None):
    """Prefill and decode a whole image; calls on_step(u, i, probs) after step i (0-based) and
    on_line_end(u, line) before every line end that is followed by another line."""
    r = np.random.default_rng(seed)
    C_, n, h, G, d = cfg.cond_len, cfg.line_width, cfg.n_lines, cfg.group, cfg.head_dim
    u = O.Unit(cfg)
    u.prefill(r.normal(size=(C_, d)), r.normal(size=(C_, d)))
    for i in range(n * h):
        _, probs = u.step(r.normal(size=(G, d)), r.normal(size=d), r.normal(size=d), want_probs=True)
        if on_step:
            on_step(u, i, probs)
        if (i + 1) % n == 0 and (i + 1) < n * h:
            if on_line_end:
                on_line_end(u, (i + 1) // n)
            u.line_end()
    return u


@pytest.mark.parametrize("G", [1, 2])
def test_accumulated_scores_are_the_decode_probabilities_summed_since_the_append(G):
    # the probabilities every step returns (Eq. 2-3, pinned to the library softmax above) are accumulated here per
    # original position; at every compressing line end the oracle's scores must be those sums / (n G), and an evicted
    # entry must never come back
    cfg = O.make_cfg(3, 4, 9, 4, 2, 1, G, 8, score_norm=2)
    mass = {}
    seen_compressions = [0]

    def on_step(u, i, probs):
        for s, p in enumerate(u.positions()):
            mass[int(p)] = mass.get(int(p), 0.0) + float(probs[:, s].sum())

    def on_line_end(u, line):
        if u.line_end_due() == 1:
            S, mid_pos = u.mid_scores()
            expect = np.array([mass[int(p)] for p in mid_pos]) / (cfg.line_width * G)
            np.testing.assert_allclose(S, expect, rtol=1e-12, atol=1e-15)
            seen_compressions[0] += 1

    _drive_generation(cfg, 11, on_step, on_line_end)
    assert seen_compressions[0] == cfg.n_lines - cfg.budget_lines


def test_accumulated_scores_are_the_sum_over_lines_of_the_cache_normalised_scores():
    # another route to the same numbers: at the end of every line (compressing or not) the cache-normalised form of
    # Eq. 9 (pinned to the library softmax with a causal cut above), taken over ALL live entries, gives each entry's
    # mean probability over that line; summed over the lines an entry has lived through this is its accumulated score
    cfg = O.make_cfg(2, 3, 8, 4, 3, 1, 2, 8, score_norm=2)
    n, G = cfg.line_width, cfg.group
    total = {}
    checked = [0]
    guide = []

    def on_step(u, i, probs):
        pass

    r = np.random.default_rng(23)
    C_, h, d = cfg.cond_len, cfg.n_lines, cfg.head_dim
    u = O.Unit(cfg)
    Ks = {}
    kc = r.normal(size=(C_, d))
    u.prefill(kc, r.normal(size=(C_, d)))
    for j in range(C_):
        Ks[j] = kc[j].astype(np.float32).astype(np.float64)
    for i in range(n * h):
        q, k = r.normal(size=(G, d)), r.normal(size=d)
        u.step(q, k, r.normal(size=d))
        Ks[C_ + i] = k.astype(np.float32).astype(np.float64)
        guide.append(q.astype(np.float32).astype(np.float64))
        if (i + 1) % n == 0 and (i + 1) < n * h:
            pos = u.positions()
            K = np.stack([Ks[int(p)] for p in pos])
            S_line = O.saliency_cache(np.stack(guide[-n:]), K, pos, C_ + i + 1 - n, list(range(len(pos))),
                                      1.0 / np.sqrt(d))
            for s, p in enumerate(pos):
                total[int(p)] = total.get(int(p), 0.0) + float(S_line[s])
            if u.line_end_due() == 1:
                S, mid_pos = u.mid_scores()
                np.testing.assert_allclose(S, [total[int(p)] for p in mid_pos], rtol=1e-10, atol=1e-14)
                checked[0] += 1
            u.line_end()
    assert checked[0] == h - cfg.budget_lines


def test_accumulated_attention_mass_is_conserved():
    # every step hands out exactly one unit of probability per head: the mass on the live entries plus the mass the
    # evicted entries took with them is G times the number of steps
    cfg = O.make_cfg(4, 5, 7, 3, 5, 1, 3, 8, score_norm=2)
    gone = [0.0]
    state = {}

    def on_line_end(u, line):
        state["before"] = dict(zip((int(p) for p in u.positions()), u.accumulated()))

    def on_step(u, i, probs):
        if "before" in state and (i % cfg.line_width) == 0 and i > 0:
            live = set(int(p) for p in u.positions())
            gone[0] += sum(a for p, a in state.pop("before").items() if p not in live)
        assert abs(u.accumulated().sum() + gone[0] - cfg.group * (i + 1)) < 1e-9

    u = _drive_generation(cfg, 31, on_step, on_line_end)
    assert gone[0] > 0.0 and u.len == cfg.cond_len + cfg.budget_lines * cfg.line_width


def test_accumulated_scoring_keeps_a_heavy_hitter_that_the_line_scores_would_drop():
    # one early key attracts every query of the first lines and none of the last line before the first compression:
    # its accumulated score is the largest of the mid region, its Eq. 9 score among the smallest
    cfgs = {sn: O.make_cfg(0, 4, 8, 5, 4, 1, 1, 4, scale=1.0, score_norm=sn) for sn in (0, 2)}
    kept = {}
    for sn, cfg in cfgs.items():
        u = O.Unit(cfg)
        u.prefill(np.zeros((0, 4)), np.zeros((0, 4)))
        n = cfg.line_width
        for i in range(cfg.budget_lines * n):
            k = np.zeros(4)
            k[1] = 0.01 * i                                # distinct, weak keys
            if i == 5:
                k[0] = 6.0                                 # the heavy hitter: visual token 6, in the mid region
            q = np.array([1.0, 0.0, 0.0, 0.0]) if i < (cfg.budget_lines - 1) * n else np.array([-1.0, 1.0, 0.0, 0.0])
            u.step(q[None, :], k, np.zeros(4))
            if (i + 1) % n == 0 and (i + 1) < cfg.budget_lines * n:
                assert u.line_end() is None
        res = u.line_end()
        kept[sn] = 5 not in set(int(p) for p in res["evicted_pos"])
    assert kept[2] and not kept[0]
