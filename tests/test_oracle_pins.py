"""Pins for the CPU checker: it is compared with things other than itself.

Each test states what fixes the expected value: the definitions in exact
rational arithmetic, textbook soft-max attention written with numpy over the
full token history, a library attention routine, an order-preserving
restatement of Algorithm 1, or an invariance the mathematics gives.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle.tova_oracle import OracleCache

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_3slot.txt")


# ----------------------------------------------------------------------------
# helpers written independently of the checker
# ----------------------------------------------------------------------------
def softmax64(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def attend_over_positions(hist_q, hist_k, hist_v, t, rows, scale, G):
    """Textbook attention of token t's query over the tokens listed in `rows`
    (original positions), from the full history; float64.
    Returns (out [H,D], probs [H,len(rows)])."""
    q = hist_q[t].astype(np.float64)                         # [H,D]
    K = np.stack([hist_k[p] for p in rows]).astype(np.float64)   # [n,Hkv,D]
    V = np.stack([hist_v[p] for p in rows]).astype(np.float64)
    H = q.shape[0]
    out = np.zeros_like(q)
    probs = np.zeros((H, len(rows)))
    for h in range(H):
        s = scale * K[:, h // G, :] @ q[h]
        p = softmax64(s)
        probs[h] = p
        out[h] = p @ V[:, h // G, :]
    return out, probs


def random_stream(seed, T, H, Hkv, D, std=1.0):
    g = np.random.default_rng(seed)
    return (g.standard_normal((T, H, D)) * std, g.standard_normal((T, Hkv, D)) * std,
            g.standard_normal((T, Hkv, D)))


def parse_golden():
    toks, steps = {}, []
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "token":
            toks[int(f[1])] = tuple(int(x) for x in f[2:6])
        elif f[0] == "step":
            steps.append((int(f[1]), int(f[2]), [int(x) for x in f[3].split(",")],
                          Fraction(f[4]), Fraction(f[5])))
    return toks, steps


# ----------------------------------------------------------------------------
# 1. hand-worked example (exact rational arithmetic fixes the fixture;
#    the checker must reproduce it, including the exact tie and self-eviction)
# ----------------------------------------------------------------------------
def test_golden_example_is_consistent_in_exact_arithmetic():
    toks, steps = parse_golden()
    cap = 3
    rows = []                                   # positions by slot
    for (t, ev, rows_after, o0, o1) in steps:
        cand = rows + [t]
        outs, probs = [], []
        for h in range(2):
            a = [Fraction(toks[p][2 * h]) for p in cand]
            v = [Fraction(toks[p][2 * h + 1]) for p in cand]
            tot = sum(a)
            p_h = [x / tot for x in a]
            probs.append(p_h)
            outs.append(sum(pp * vv for pp, vv in zip(p_h, v)))
        assert outs == [o0, o1], t
        if len(cand) <= cap:
            rows = cand
            assert ev == -1
        else:
            mean = [(probs[0][j] + probs[1][j]) / 2 for j in range(len(cand))]
            j = min(range(len(cand)), key=lambda i: (mean[i], i))
            assert cand[j] == ev, t
            if j < cap:
                rows[j] = t
        assert rows + [-1] * (cap - len(rows)) == rows_after, t


@pytest.mark.parametrize("precision", ["f32", "f64"])
@pytest.mark.parametrize("D", [1, 64])
def test_checker_reproduces_golden_example(precision, D):
    toks, steps = parse_golden()
    c = OracleCache(1, 2, 2, D, 3, sm_scale=1.0, precision=precision)
    for (t, ev, rows_after, o0, o1) in steps:
        q = np.zeros((1, 2, D)); q[..., 0] = 1.0
        k = np.zeros((1, 2, D)); v = np.zeros((1, 2, D))
        a0, v0, a1, v1 = toks[t]
        k[0, 0, 0], k[0, 1, 0] = np.log(a0), np.log(a1)
        v[0, 0, 0], v[0, 1, 0] = v0, v1
        out, evp, victim, argmin, gap, _ = c.step(q, k, v, t)
        assert evp[0] == ev, t
        assert list(c.pos[0]) == rows_after, t
        tol = 2e-5 if precision == "f32" else 1e-12
        assert abs(out[0, 0, 0] - float(o0)) < tol and abs(out[0, 1, 0] - float(o1)) < tol
        assert np.all(out[0, :, 1:] == 0)


# ----------------------------------------------------------------------------
# 2. brute force on tiny states: outputs, head-averaged weights and the victim
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("H,Hkv,D,cap,T", [(1, 1, 4, 1, 9), (2, 2, 3, 2, 12), (4, 2, 8, 5, 40),
                                           (6, 2, 16, 8, 60), (4, 4, 64, 7, 30)])
@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_brute_force_tiny(H, Hkv, D, cap, T, precision):
    q, k, v = random_stream(100 + cap, T, H, Hkv, D)
    scale = 0.37
    c = OracleCache(1, H, Hkv, D, cap, sm_scale=scale, precision=precision)
    rows = []
    tol = 3e-5 if precision == "f32" else 1e-12
    for t in range(T):
        out, evp, victim, argmin, gap, mean = c.step(q[t][None], k[t][None], v[t][None], t, want_mean=True)
        cand = rows + [t]
        ref_out, probs = attend_over_positions(q, k, v, t, cand, scale, H // Hkv)
        assert np.abs(out[0] - ref_out).max() < tol
        if len(cand) <= cap:
            assert evp[0] == -1 and victim[0] == -1
            rows = cand
        else:
            ref_mean = probs.mean(axis=0)
            assert np.abs(mean[0, :len(cand)] - ref_mean).max() < tol
            j = int(victim[0])
            assert argmin[0] == j and gap[0] == 0
            # the dropped row attains the brute-force minimum (up to rounding)
            assert ref_mean[j] - ref_mean.min() < tol
            assert evp[0] == cand[j]
            if j < cap:
                rows[j] = t
        assert list(c.pos[0, :len(rows)]) == rows
        assert c.len[0] == min(t + 1, cap)                      # g(t) = min(t, k), Section 3.3


# ----------------------------------------------------------------------------
# 3. capacity >= stream length: the bounded state is the unbounded one and the
#    outputs are plain causal attention (library routine)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("H,Hkv,D,T", [(4, 4, 16, 24), (8, 2, 32, 33)])
@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_unbounded_equals_library_causal_attention(H, Hkv, D, T, precision):
    q, k, v = random_stream(7, T, H, Hkv, D)
    tdt = torch.float32 if precision == "f32" else torch.float64
    scale = 1.0 / np.sqrt(D)
    c = OracleCache(1, H, Hkv, D, T + 3, precision=precision)
    outs = []
    for t in range(T):
        out, evp, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        assert evp[0] == -1
        outs.append(out[0])
    outs = np.stack(outs)                                           # [T,H,D]
    G = H // Hkv
    tq = torch.tensor(q, dtype=tdt).permute(1, 0, 2)[None]          # [1,H,T,D]
    tk = torch.tensor(np.repeat(k, G, axis=1), dtype=tdt).permute(1, 0, 2)[None]
    tv = torch.tensor(np.repeat(v, G, axis=1), dtype=tdt).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    ref = ref[0].permute(1, 0, 2).numpy()
    tol = 2e-5 if precision == "f32" else 1e-12
    assert np.abs(outs - ref).max() < tol
    assert list(c.pos[0, :T]) == list(range(T)) and c.len[0] == T


def test_first_token_output_is_its_value():
    q, k, v = random_stream(3, 1, 4, 2, 8)
    c = OracleCache(1, 4, 2, 8, 4, precision="f32")
    out, *_ = c.step(q[0][None], k[0][None], v[0][None], 0)
    assert np.array_equal(out[0], np.repeat(v[0], 2, axis=0).astype(np.float32))


# ----------------------------------------------------------------------------
# 4. Algorithm 1 restated with an order-preserving (concatenating) cache:
#    same retained position sets and outputs on tie-free inputs
# ----------------------------------------------------------------------------
def alg1_stream(q, k, v, cap, scale, G):
    """Append, attend, then drop by deleting the row (rows stay in position
    order).  Returns per step (set of retained positions, out)."""
    kc = np.zeros((q.shape[1], 0, q.shape[2]))       # [attn_heads, num_kv, D]
    vc = np.zeros_like(kc)
    kept, res = [], []
    for t in range(q.shape[0]):
        kc = np.concatenate([kc, np.repeat(k[t], G, axis=0)[:, None, :]], axis=1)
        vc = np.concatenate([vc, np.repeat(v[t], G, axis=0)[:, None, :]], axis=1)
        kept.append(t)
        w = softmax64(scale * np.einsum("hd,hnd->hn", q[t], kc))     # last query's weights
        out = np.einsum("hn,hnd->hd", w, vc)
        if kc.shape[1] > cap:
            i = int(np.argmin(w.mean(axis=0)))
            kc = np.concatenate([kc[:, :i], kc[:, i + 1:]], axis=1)
            vc = np.concatenate([vc[:, :i], vc[:, i + 1:]], axis=1)
            del kept[i]
        res.append((set(kept), out))
    return res


@pytest.mark.parametrize("H,Hkv,D,cap,T", [(4, 4, 8, 6, 80), (8, 2, 16, 16, 120)])
def test_matches_order_preserving_algorithm1(H, Hkv, D, cap, T):
    q, k, v = random_stream(11, T, H, Hkv, D)
    scale = 1.0 / np.sqrt(D)
    ref = alg1_stream(q, k, v, cap, scale, H // Hkv)
    c = OracleCache(1, H, Hkv, D, cap, precision="f64")
    for t in range(T):
        out, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        assert set(c.pos[0, :c.len[0]].tolist()) == ref[t][0], t
        assert np.abs(out[0] - ref[t][1]).max() < 1e-12


# ----------------------------------------------------------------------------
# 5. invariances
# ----------------------------------------------------------------------------
def test_slot_permutation_changes_nothing():
    H, Hkv, D, cap, T = 4, 2, 8, 6, 30
    q, k, v = random_stream(5, T, H, Hkv, D)
    a = OracleCache(1, H, Hkv, D, cap, precision="f64")
    b = OracleCache(1, H, Hkv, D, cap, precision="f64")
    g = np.random.default_rng(0)
    for t in range(T):
        if t >= cap:                         # shuffle b's rows before every step
            perm = g.permutation(cap)
            b.K[:] = b.K[:, :, perm]; b.V[:] = b.V[:, :, perm]; b.pos[:] = b.pos[:, perm]
        oa, ea, *_ = a.step(q[t][None], k[t][None], v[t][None], t)
        ob, eb, *_ = b.step(q[t][None], k[t][None], v[t][None], t)
        assert ea[0] == eb[0]
        assert np.abs(oa - ob).max() < 1e-12
        assert set(a.pos[0].tolist()) == set(b.pos[0].tolist())


def test_constant_logit_shift_per_head_changes_nothing():
    """An extra component (q: c_h, every key: 1) adds c_h*scale to all logits of
    head h; soft-max, outputs and victims do not move."""
    H, Hkv, D, cap, T = 4, 4, 8, 5, 40
    q, k, v = random_stream(9, T, H, Hkv, D)
    shift = np.array([3.0, -2.0, 0.5, 7.0])
    q2 = np.concatenate([q, np.broadcast_to(shift[None, :, None], (T, H, 1))], axis=2)
    k2 = np.concatenate([k, np.ones((T, Hkv, 1))], axis=2)
    v2 = np.concatenate([v, np.zeros((T, Hkv, 1))], axis=2)
    a = OracleCache(1, H, Hkv, D, cap, sm_scale=0.4, precision="f64")
    b = OracleCache(1, H, Hkv, D + 1, cap, sm_scale=0.4, precision="f64")
    for t in range(T):
        oa, ea, *_ = a.step(q[t][None], k[t][None], v[t][None], t)
        ob, eb, *_ = b.step(q2[t][None], k2[t][None], v2[t][None], t)
        assert ea[0] == eb[0]
        assert np.abs(oa - ob[..., :D]).max() < 1e-10


def test_single_head_is_per_head_tova():
    """With one head the layer average is that head's weights (Section 4)."""
    D, cap, T = 8, 4, 30
    q, k, v = random_stream(13, T, 1, 1, D)
    c = OracleCache(1, 1, 1, D, cap, sm_scale=1.0, precision="f64")
    rows = []
    for t in range(T):
        cand = rows + [t]
        _, probs = attend_over_positions(q, k, v, t, cand, 1.0, 1)
        out, evp, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        if len(cand) <= cap:
            rows = cand
        else:
            j = int(np.argmin(probs[0]))
            assert evp[0] == cand[j]
            if j < cap:
                rows[j] = t


def test_sequences_are_independent():
    H, Hkv, D, cap, T, B = 4, 2, 8, 5, 25, 3
    streams = [random_stream(20 + b, T, H, Hkv, D) for b in range(B)]
    batched = OracleCache(B, H, Hkv, D, cap, precision="f32", threads=2)
    singles = [OracleCache(1, H, Hkv, D, cap, precision="f32", threads=1) for _ in range(B)]
    for t in range(T):
        qb = np.stack([s[0][t] for s in streams]); kb = np.stack([s[1][t] for s in streams])
        vb = np.stack([s[2][t] for s in streams])
        ob, eb, *_ = batched.step(qb, kb, vb, t)
        for b in range(B):
            o1, e1, *_ = singles[b].step(qb[b][None], kb[b][None], vb[b][None], t)
            assert np.array_equal(o1[0], ob[b]) and e1[0] == eb[b]
    for b in range(B):
        assert np.array_equal(singles[b].pos[0], batched.pos[b])
        assert np.array_equal(singles[b].K[0], batched.K[b])


def test_forced_victim_and_gap():
    H, Hkv, D, cap = 2, 2, 4, 3
    q, k, v = random_stream(31, 5, H, Hkv, D)
    a = OracleCache(1, H, Hkv, D, cap, precision="f64")
    b = OracleCache(1, H, Hkv, D, cap, precision="f64")
    for t in range(3):
        a.step(q[t][None], k[t][None], v[t][None], t)
        b.step(q[t][None], k[t][None], v[t][None], t)
    _, ea, va, aa, ga, mean = a.step(q[3][None], k[3][None], v[3][None], 3, want_mean=True)
    other = (int(va[0]) + 1) % (cap + 1)
    _, eb, vb, ab, gb, _ = b.step(q[3][None], k[3][None], v[3][None], 3, forced=np.array([other]))
    assert vb[0] == other and ab[0] == va[0]
    assert abs(gb[0] - (mean[0, other] - mean[0].min())) < 1e-15 and gb[0] > 0
    expect = list(range(3))
    if other < cap:
        expect[other] = 3
    assert list(b.pos[0]) == expect


# ----------------------------------------------------------------------------
# 6. float checker against the double one; the memory model against Table 1
# ----------------------------------------------------------------------------
def test_float_build_tracks_double_build():
    from paper_2401_06104_b200 import workloads as W
    w = W.WORKLOADS["llama2_7b_layer"].scaled(batch=2, n_q_heads=8, n_kv_heads=8, capacity=48)
    a = OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, precision="f32")
    b = OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, precision="f64")
    for t in range(160):
        q, k, v = W.token(w, t)
        oa, ea, va, *_ = a.step(q, k, v, t)
        ob, eb, vb, ab, gb, _ = b.step(q, k, v, t, forced=va)
        assert np.abs(oa - ob).max() < 1e-5
        assert np.all(gb < 1e-6)                 # any disagreement is a near tie
        assert np.array_equal(ea, eb) and np.array_equal(a.pos, b.pos)


def test_memory_model_matches_table_1():
    """Table 1, first row: KV memory of LLaMA-2-7B in bf16 at batch 1."""
    per_token = 2 * 32 * 32 * 128 * 2            # K and V, 32 layers, 32 heads, 128 dims, 2 bytes
    printed = {256: 0.15, 512: 0.28, 1024: 0.56, 2048: 1.11, 4096: 2.18}
    for size, gb in printed.items():
        assert abs(per_token * size / 1e9 - gb) / gb < 0.11
    from paper_2401_06104_b200 import workloads as W
    w = W.WORKLOADS["llama2_7b_layer"]
    assert w.step_bytes() == 8 * (per_token // 32) * 512 + 8 * (per_token // 32)


# ----------------------------------------------------------------------------
# 9. the other compression policies: Window, Window+i, TOVA+i (Section 4.1 and
#    the appendix ablation)
# ----------------------------------------------------------------------------
POLICY_GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_3slot_policies.txt")


def parse_policy_golden():
    traces, cur = [], None
    for line in open(POLICY_GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "trace":
            cur = (f[1], int(f[2]), [])
            traces.append(cur)
        elif f[0] == "step":
            cur[2].append((int(f[1]), int(f[2]), [int(x) for x in f[3].split(",")], Fraction(f[4]), Fraction(f[5])))
    return traces


def test_policy_traces_are_consistent_in_exact_arithmetic():
    """The fixture follows from the definitions in exact rational arithmetic."""
    toks, _ = parse_golden()
    cap = 3
    for policy, keep, steps in parse_policy_golden():
        rows = []
        for (t, ev, rows_after, o0, o1) in steps:
            cand = rows + [t]
            outs, probs = [], []
            for h in range(2):
                a = [Fraction(toks[p][2 * h]) for p in cand]
                v = [Fraction(toks[p][2 * h + 1]) for p in cand]
                tot = sum(a)
                probs.append([x / tot for x in a])
                outs.append(sum(x / tot * vv for x, vv in zip(a, v)))
            assert outs == [o0, o1], (policy, keep, t)
            if len(cand) <= cap:
                rows = cand
                assert ev == -1
            else:
                free = [i for i in range(len(cand)) if cand[i] >= keep]
                if policy == "window":
                    j = min(free, key=lambda i: (cand[i], i))
                else:
                    mean = [(probs[0][i] + probs[1][i]) / 2 for i in range(len(cand))]
                    j = min(free, key=lambda i: (mean[i], i))
                assert cand[j] == ev, (policy, keep, t)
                if j < cap:
                    rows[j] = t
            assert rows + [-1] * (cap - len(rows)) == rows_after, (policy, keep, t)


@pytest.mark.parametrize("precision", ["f32", "f64"])
def test_checker_reproduces_policy_traces(precision):
    toks, _ = parse_golden()
    for policy, keep, steps in parse_policy_golden():
        c = OracleCache(1, 2, 2, 1, 3, sm_scale=1.0, precision=precision, policy=policy, keep_first=keep)
        for (t, ev, rows_after, o0, o1) in steps:
            q = np.ones((1, 2, 1))
            a0, v0, a1, v1 = toks[t]
            k = np.array([[[np.log(a0)], [np.log(a1)]]])
            v = np.array([[[float(v0)], [float(v1)]]])
            out, evp, victim, argmin, gap, _ = c.step(q, k, v, t)
            assert evp[0] == ev, (policy, keep, t)
            assert list(c.pos[0]) == rows_after, (policy, keep, t)
            tol = 2e-5 if precision == "f32" else 1e-12
            assert abs(out[0, 0, 0] - float(o0)) < tol and abs(out[0, 1, 0] - float(o1)) < tol


@pytest.mark.parametrize("cap,keep,T", [(8, 0, 50), (8, 1, 50), (16, 4, 90), (5, 4, 30)])
def test_window_policy_closed_form(cap, keep, T):
    """Window(+i) keeps exactly the first i and the most recent k - i positions,
    whatever the inputs (Section 4.1); each step drops the earliest of the rest."""
    H, Hkv, D = 4, 2, 8
    q, k, v = random_stream(7, T, H, Hkv, D)
    c = OracleCache(1, H, Hkv, D, cap, precision="f64", policy="window", keep_first=keep)
    for t in range(T):
        out, evp, *_ = c.step(q[t][None], k[t][None], v[t][None], t)
        held = sorted(int(p) for p in c.pos[0] if p >= 0)
        if t + 1 <= cap:
            assert held == list(range(t + 1)) and evp[0] == -1
        else:
            assert held == list(range(keep)) + list(range(t + 1 - (cap - keep), t + 1))
            assert evp[0] == t - (cap - keep)


def test_plus_zero_is_the_plain_policy_and_protected_rows_stay():
    H, Hkv, D, cap, T = 4, 2, 16, 6, 80
    q, k, v = random_stream(11, T, H, Hkv, D, std=1.5)
    plain = OracleCache(1, H, Hkv, D, cap, precision="f64")
    plus0 = OracleCache(1, H, Hkv, D, cap, precision="f64", policy="tova", keep_first=0)
    plus3 = OracleCache(1, H, Hkv, D, cap, precision="f64", policy="tova", keep_first=3)
    rows3 = []
    scale = 1.0 / np.sqrt(D)
    for t in range(T):
        a = plain.step(q[t][None], k[t][None], v[t][None], t)
        b = plus0.step(q[t][None], k[t][None], v[t][None], t)
        assert a[1][0] == b[1][0] and np.array_equal(plain.pos, plus0.pos) and np.array_equal(a[0], b[0])
        out, evp, victim, argmin, gap, mean = plus3.step(q[t][None], k[t][None], v[t][None], t, want_mean=True)
        # brute force from the full history: textbook soft-max, mean over heads, arg-min over unprotected rows
        cand = rows3 + [t]
        ref_out, probs = attend_over_positions(q, k, v, t, cand, scale, H // Hkv)
        assert np.abs(out[0] - ref_out).max() < 1e-12
        if len(cand) <= cap:
            rows3 = cand
        else:
            ref_mean = probs.mean(axis=0)
            free = [i for i in range(len(cand)) if cand[i] >= 3]
            j = min(free, key=lambda i: (ref_mean[i], i))
            assert evp[0] == cand[j] and evp[0] >= 3
            if j < cap:
                rows3[j] = t
        assert {0, 1, 2} <= set(int(p) for p in plus3.pos[0]) or t < 2
