"""Pins for the checker's per-unit policies: TOVA-head (Section 4; appendix
ablation) and H2O, layer-wise and head-wise (Section 4.1).

As for the layer policy, the checker is compared with things other than
itself: the definitions in exact rational arithmetic on hand-worked traces,
restatements over the full token history with textbook soft-max in float64
(order-preserving lists per head), closed forms, and special cases that reduce
to a policy pinned elsewhere."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle.tova_oracle import OracleCache, OracleUnitsCache
from test_oracle_pins import attend_over_positions, parse_golden, random_stream, softmax64

GOLDEN_UNITS = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_3slot_units.txt")


def parse_unit_golden():
    traces = []
    for line in open(GOLDEN_UNITS):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "trace":
            traces.append((f[1], int(f[2]), []))
        elif f[0] == "step":
            traces[-1][2].append((int(f[1]), [int(x) for x in f[2].split(",")],
                                  [[int(x) for x in u.split(",")] for u in f[3].split(";")],
                                  Fraction(f[4]), Fraction(f[5])))
    return traces


# ----------------------------------------------------------------------------
# 1. hand-worked traces: the fixture is consistent in exact arithmetic, and the
#    checker reproduces it
# ----------------------------------------------------------------------------
def test_unit_traces_are_consistent_in_exact_arithmetic():
    toks, _ = parse_golden()
    cap = 3
    for policy, recent, steps in parse_unit_golden():
        h2o = policy.startswith("h2o")
        U = 1 if policy == "h2o_layer" else 2
        rows = [[] for _ in range(U)]           # positions by slot, per unit
        sums = [[] for _ in range(U)]           # accumulated weight by slot (H2O)
        for (t, ev, rows_after, o0, o1) in steps:
            probs, outs = [], []
            for h in range(2):
                cand = rows[0 if U == 1 else h] + [t]
                a = [Fraction(toks[p][2 * h]) for p in cand]
                v = [Fraction(toks[p][2 * h + 1]) for p in cand]
                p_h = [x / sum(a) for x in a]
                probs.append(p_h)
                outs.append(sum(pp * vv for pp, vv in zip(p_h, v)))
            assert outs == [o0, o1], (policy, recent, t)
            for u in range(U):
                cand = rows[u] + [t]
                heads = [0, 1] if U == 1 else [u]
                w = [sum(probs[h][j] for h in heads) / len(heads) for j in range(len(cand))]
                key = [s + x for s, x in zip(sums[u], w)] + [w[-1]] if h2o else w
                if len(cand) <= cap:
                    rows[u], sums[u] = cand, list(key)
                    assert ev[u] == -1
                    continue
                droppable = [j for j in range(len(cand)) if not (h2o and t - cand[j] < recent)]
                j = min(droppable, key=lambda i: (key[i], i))
                assert cand[j] == ev[u], (policy, recent, t, u)
                sums[u] = list(key[:-1])
                if j < cap:
                    rows[u][j] = t
                    sums[u][j] = key[-1]
                assert rows[u] == rows_after[u], (policy, recent, t, u)


@pytest.mark.parametrize("precision", ["f32", "f64"])
@pytest.mark.parametrize("D", [1, 64])
def test_checker_reproduces_unit_traces(precision, D):
    toks, _ = parse_golden()
    for policy, recent, steps in parse_unit_golden():
        c = OracleUnitsCache(1, 2, 2, D, 3, policy, recent=recent, sm_scale=1.0, precision=precision)
        for (t, ev, rows_after, o0, o1) in steps:
            q = np.zeros((1, 2, D)); q[..., 0] = 1.0
            k = np.zeros((1, 2, D)); v = np.zeros((1, 2, D))
            a0, v0, a1, v1 = toks[t]
            k[0, 0, 0], k[0, 1, 0] = np.log(a0), np.log(a1)
            v[0, 0, 0], v[0, 1, 0] = v0, v1
            out, evp, *_ = c.step(q, k, v, t)
            assert evp[0].tolist() == ev, (policy, recent, t)
            assert c.pos[0].tolist() == rows_after, (policy, recent, t)
            tol = 2e-5 if precision == "f32" else 1e-12
            assert abs(out[0, 0, 0] - float(o0)) < tol and abs(out[0, 1, 0] - float(o1)) < tol


def test_traces_show_heads_keeping_different_tokens():
    """The point of the head-wise policies: at t=3 the two heads drop different
    positions, both different from the layer policy's choice (position 2)."""
    for policy, recent, steps in parse_unit_golden():
        if policy == "tova_head":
            t3 = steps[3]
            assert t3[1] == [1, 0] and t3[2][0] != t3[2][1]


# ----------------------------------------------------------------------------
# 2. restatement over the full history: order-preserving lists per unit,
#    textbook soft-max in float64, accumulated scores recomputed from the history
# ----------------------------------------------------------------------------
def history_policy(q, k, v, cap, scale, H, Hkv, policy, recent):
    """Per unit a list of retained positions in position order (rows are deleted, as in Algorithm 1's
    concatenation).  H2O scores are not carried: every step recomputes, for each retained position, the sum
    of its weights over all the steps since it entered, from stored per-step weights.
    Returns per step (retained sets per unit, out [H,D])."""
    G = H // Hkv
    U = 1 if policy == "h2o_layer" else Hkv
    h2o = policy.startswith("h2o")
    kept = [[] for _ in range(U)]
    weight_log = [dict() for _ in range(U)]      # unit -> {position: [weights it received, step by step]}
    res = []
    for t in range(q.shape[0]):
        out = np.zeros((H, q.shape[2]))
        probs = {}
        for h in range(H):
            u = 0 if U == 1 else h // G
            cand = kept[u] + [t]
            o, p = attend_over_positions(q, k, v, t, cand, scale, G)   # all heads; keep this head's row
            out[h] = o[h]
            probs[h] = p[h]
        for u in range(U):
            cand = kept[u] + [t]
            heads = range(H) if U == 1 else range(u * G, (u + 1) * G)
            w = np.mean([probs[h] for h in heads], axis=0)
            for j, p_ in enumerate(cand):
                weight_log[u].setdefault(p_, []).append(w[j])
            if len(cand) > cap:
                if h2o:
                    droppable = [j for j, p_ in enumerate(cand) if t - p_ >= recent]
                    total = [sum(weight_log[u][cand[j]]) for j in droppable]
                    j = droppable[int(np.argmin(total))]
                else:
                    j = int(np.argmin(w))
                del weight_log[u][cand[j]]
                del cand[j]
            kept[u] = cand
        res.append(([set(x) for x in kept], out))
    return res


@pytest.mark.parametrize("policy,recent", [("tova_head", 0), ("h2o_layer", 0), ("h2o_head", 0), ("h2o_layer", 2),
                                           ("h2o_head", 5)])
@pytest.mark.parametrize("H,Hkv,D,cap,T", [(4, 4, 8, 6, 70), (8, 2, 16, 12, 90), (2, 1, 4, 3, 40)])
def test_matches_history_restatement(policy, recent, H, Hkv, D, cap, T):
    q, k, v = random_stream(21 + cap, T, H, Hkv, D)
    scale = 1.0 / np.sqrt(D)
    recent = min(recent, cap)
    rec = recent or cap - cap // 2
    ref = history_policy(q, k, v, cap, scale, H, Hkv, policy, rec)
    c = OracleUnitsCache(1, H, Hkv, D, cap, policy, recent=recent, precision="f64")
    for t in range(T):
        out, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        n = int(c.len[0])
        assert n == min(t + 1, cap)                       # g(t) = min(t, k), Section 3.3
        got = [set(c.pos[0, u, :n].tolist()) for u in range(c.U)]
        assert got == ref[t][0], (t, got, ref[t][0])
        assert np.abs(out[0] - ref[t][1]).max() < 1e-12


# ----------------------------------------------------------------------------
# 3. special cases that reduce to something pinned elsewhere, closed forms
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("D,cap,T", [(8, 5, 60), (16, 9, 50)])
def test_one_head_makes_the_head_policy_the_layer_policy(D, cap, T):
    q, k, v = random_stream(31, T, 1, 1, D)
    layer = OracleCache(1, 1, 1, D, cap, precision="f64")
    head = OracleUnitsCache(1, 1, 1, D, cap, "tova_head", precision="f64")
    hl = OracleUnitsCache(1, 1, 1, D, cap, "h2o_layer", precision="f64")
    hh = OracleUnitsCache(1, 1, 1, D, cap, "h2o_head", precision="f64")
    for t in range(T):
        a = layer.step(q[t][None], k[t][None], v[t][None], t)
        b = head.step(q[t][None], k[t][None], v[t][None], t)
        c = hl.step(q[t][None], k[t][None], v[t][None], t)
        d = hh.step(q[t][None], k[t][None], v[t][None], t)
        assert a[1][0] == b[1][0, 0] and np.array_equal(a[0], b[0])
        assert np.array_equal(layer.pos[0], head.pos[0, 0])
        assert np.array_equal(c[1], d[1]) and np.array_equal(c[0], d[0]) and np.array_equal(hl.acc, hh.acc)


@pytest.mark.parametrize("policy", ["h2o_layer", "h2o_head"])
def test_window_as_large_as_the_state_is_first_in_first_out(policy):
    """recent = k: only the oldest candidate is outside the window, so H2O is the Window policy:
    the state holds the k most recent positions (closed form), whatever the scores."""
    H, Hkv, D, cap, T = 4, 2, 8, 7, 50
    q, k, v = random_stream(41, T, H, Hkv, D)
    c = OracleUnitsCache(1, H, Hkv, D, cap, policy, recent=cap, precision="f64")
    w = OracleCache(1, H, Hkv, D, cap, precision="f64", policy="window")
    for t in range(T):
        out, ev, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        ow, ew, *_ = w.step(q[t][None], k[t][None], v[t][None], t)
        assert np.all(ev[0] == ew[0])
        assert np.abs(out - ow).max() < 1e-12
        for u in range(c.U):
            assert sorted(p for p in c.pos[0, u].tolist() if p >= 0) == list(range(max(0, t + 1 - cap), t + 1))


@pytest.mark.parametrize("policy", ["h2o_layer", "h2o_head"])
def test_accumulated_scores_are_column_sums_of_the_causal_attention_matrix(policy):
    """While nothing is dropped (capacity >= T) the score of token j after step t is the sum over
    queries j..t of the (head-averaged) causal soft-max weight on j: textbook matrix, float64."""
    H, Hkv, D, T = 4, 2, 8, 24
    G = H // Hkv
    q, k, v = random_stream(51, T, H, Hkv, D)
    scale = 0.3
    c = OracleUnitsCache(1, H, Hkv, D, T, policy, precision="f64", sm_scale=scale)
    A = np.zeros((H, T, T))
    for h in range(H):
        s = scale * q[:, h, :] @ k[:, h // G, :].T
        s[np.triu_indices(T, 1)] = -np.inf
        A[h] = softmax64(s)
    for t in range(T):
        c.step(q[t][None], k[t][None], v[t][None], t)
        for u in range(c.U):
            heads = range(H) if c.U == 1 else range(u * G, (u + 1) * G)
            col = np.mean([A[h, :t + 1, :t + 1].sum(axis=0) for h in heads], axis=0)
            assert np.abs(c.acc[0, u, :t + 1] - col).max() < 1e-12


@pytest.mark.parametrize("policy", ["h2o_layer", "h2o_head"])
def test_recent_window_is_never_touched(policy):
    H, Hkv, D, cap, T = 4, 4, 8, 10, 80
    q, k, v = random_stream(61, T, H, Hkv, D)
    c = OracleUnitsCache(1, H, Hkv, D, cap, policy, precision="f32")       # recent = 5
    for t in range(T):
        _, ev, victim, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        for u in range(c.U):
            held = set(c.pos[0, u].tolist())
            assert set(range(max(0, t - 4), t + 1)) <= held
            assert ev[0, u] == -1 or t - ev[0, u] >= 5


def test_forced_victim_and_gap_for_units():
    H, Hkv, D, cap = 4, 2, 8, 6
    q, k, v = random_stream(71, cap + 1, H, Hkv, D)
    a = OracleUnitsCache(1, H, Hkv, D, cap, "tova_head", precision="f64")
    b = OracleUnitsCache(1, H, Hkv, D, cap, "tova_head", precision="f64")
    for t in range(cap):
        a.step(q[t][None], k[t][None], v[t][None], t)
        b.step(q[t][None], k[t][None], v[t][None], t)
    _, ev, victim, argmin, gap, score = a.step(q[cap][None], k[cap][None], v[cap][None], cap, want_score=True)
    assert np.all(victim == argmin) and np.all(gap == 0)
    forced = (argmin[0] + 1) % (cap + 1)
    _, ev2, victim2, argmin2, gap2, _ = b.step(q[cap][None], k[cap][None], v[cap][None], cap, forced=forced[None])
    assert np.array_equal(victim2[0], forced) and np.array_equal(argmin2, argmin)
    for u in range(Hkv):
        assert abs(gap2[0, u] - (score[0, u, forced[u]] - score[0, u, argmin[0, u]])) < 1e-15


def test_sequences_are_independent_for_units():
    H, Hkv, D, cap, T, B = 4, 2, 8, 5, 30, 3
    streams = [random_stream(80 + b, T, H, Hkv, D) for b in range(B)]
    full = OracleUnitsCache(B, H, Hkv, D, cap, "h2o_head", precision="f32", threads=2)
    ones = [OracleUnitsCache(1, H, Hkv, D, cap, "h2o_head", precision="f32") for _ in range(B)]
    for t in range(T):
        q, k, v = (np.stack([s[i][t] for s in streams]) for i in range(3))
        of, ef, *_ = full.step(q, k, v, t)
        for b in range(B):
            o1, e1, *_ = ones[b].step(q[b][None], k[b][None], v[b][None], t)
            assert np.array_equal(o1[0], of[b]) and np.array_equal(e1[0], ef[b])
