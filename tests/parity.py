"""Lock-step comparison of the CUDA library with the CPU checker.

Both sides consume the same seeded tokens.  The GPU runs blocks of tokens
through the C ABI (tova_prefill or tova_decode_step); the checker replays every
token.  Rule for the victim: the checker is told which candidate the GPU
dropped and reports how far that candidate's head-averaged weight lies above
the minimum; a gap below 1e-6 is accepted (either choice is right when the two
lowest averages are that close) and the checker follows the GPU's choice,
otherwise the test fails at that token.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

import paper_2401_06104_b200 as tova
from paper_2401_06104_b200 import workloads as W
from oracle.tova_oracle import OracleCache

GAP_TOL = 1e-6
# A disagreement about the victim is only explained by rounding when the two candidates' averages differ by
# rounding-level amounts RELATIVE to their size: both sides evaluate a soft-max weight to within a few 1e-6 of its
# value (fp32 dot products in different orders, exp versus exp2), and at states of thousands of rows the lowest
# averages are 1e-5 and less, where the absolute 1e-6 alone would accept almost any candidate near the bottom.
REL_GAP_TOL = 1e-4


def hand_tol(expected: float) -> float:
    """Tolerance for fp32 outputs of hand-worked examples: 1e-5, or 4 units in the last place where the value is so
    large (beyond 32: one ulp is 3.8e-6) that 1e-5 would be under three ulps.  The GPU's weights are exp2 of
    log2(e)-scaled logits normalised by a reciprocal; each is within about 3e-7 of its value, and an output near 36
    that averages values up to 56 inherits up to ~1e-5 of that."""
    return max(1e-5, 4.0 * float(np.spacing(np.float32(abs(expected)))))


def out_tol(w: W.Workload) -> float:
    """Max-abs tolerance on attention outputs: 2e-3 for bf16 inputs with fp32
    accumulation, 1e-5 for fp32 inputs."""
    return 2e-3 if w.dtype == W.DTYPE_BF16 else 1e-5


@dataclass
class ParityReport:
    steps: int = 0
    evictions: int = 0
    resyncs: int = 0            # checker's own arg-min differed (gap < 1e-6)
    self_evictions: int = 0
    max_err: float = 0.0
    max_gap: float = 0.0
    max_rel_gap: float = 0.0    # largest gap / lowest average among the resyncs
    evicted_log: List[np.ndarray] = field(default_factory=list)


POLICIES = {"tova": tova.TOVA_POLICY_TOVA, "window": tova.TOVA_POLICY_WINDOW,
            "tova_head": tova.TOVA_POLICY_TOVA_HEAD, "h2o_layer": tova.TOVA_POLICY_H2O_LAYER,
            "h2o_head": tova.TOVA_POLICY_H2O_HEAD}


def make_cache(w: W.Workload, sm_scale: float = 0.0, evict: bool = True, chunk_rows: int = 0,
               fused_merge: bool = True, policy: str = "tova", keep_first: int = 0, prefill_ws: bool = False,
               chunk_cluster: int = 0, rope_base: float = 0.0, chunk_barriers: int = 0):
    c = tova.TovaCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, dtype=w.dtype,
                       sm_scale=sm_scale, evict=evict)
    if chunk_rows:
        c.tova_cache_set_chunk_rows(chunk_rows)
    if not fused_merge:
        c.tova_cache_set_fused_merge(False)
    if policy != "tova" or keep_first:
        c.tova_cache_set_policy(POLICIES[policy], keep_first)
    if rope_base:                        # position compression: q and k come without rotary embedding
        c.tova_cache_set_position_compression(rope_base)
    if prefill_ws:                       # prompt tokens that meet a full state go in chunks of up to 64
        c.tova_cache_set_prefill_workspace()
        if chunk_cluster:
            c.tova_cache_set_chunk_cluster(chunk_cluster)
        if chunk_barriers:
            c.tova_cache_set_chunk_barriers(chunk_barriers)
    return c


def gpu_block(cache, w: W.Workload, q, k, v, first_pos: int, use_prefill: bool = True):
    """Run a block of tokens on the GPU; returns (out [T,B,H,D], evicted [T,B]) on the host."""
    T = q.shape[0]
    dq, dk, dv = (tova.to_device(a, w.dtype) for a in (q, k, v))
    out = torch.empty(T, w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda:0")
    ev = torch.full((T, w.batch), -12345, dtype=torch.int32, device="cuda:0")
    if use_prefill:
        cache.tova_prefill(dq, dk, dv, T, first_pos, out, ev)
    else:
        for t in range(T):
            cache.tova_decode_step(dq[t], dk[t], dv[t], first_pos + t, out[t], ev[t])
    torch.cuda.synchronize()
    return out.cpu().numpy(), ev.cpu().numpy()


def run_lockstep(w: W.Workload, n_tokens: int, *, seqs: Optional[Sequence[int]] = None,
                 block: int = 64, use_prefill: bool = True, chunk_rows: int = 0,
                 sm_scale: float = 0.0, layer: int = 0, cache=None, oracle=None,
                 first_pos: int = 0, check_state_every: int = 4, direct_fill: bool = False,
                 fused_merge: bool = True, policy: str = "tova", keep_first: int = 0,
                 period: int = 0, prefill_ws: bool = False, chunk_cluster: int = 0,
                 rope_base: float = 0.0, chunk_barriers: int = 0) -> ParityReport:
    """Feed n_tokens tokens to both sides and compare at every token.

    direct_fill: while the state is filling nothing is dropped (Section 3.3), so
    the checker's state after the first `capacity` tokens is those tokens in
    order; it is then written from the generated tokens instead of replayed, and
    only the slot table is compared for that phase (the checker's cost per
    token grows with the state; this keeps capacity-4096 cases affordable).

    period > 0: the token at position p carries the generator's (q, k, v) of
    position p mod period (drawing thousands of distinct tokens for a batch of 64
    takes minutes); repeated keys give exactly equal averages, which the
    lowest-slot rule must then resolve the same way on both sides."""
    seqs = list(range(w.batch)) if seqs is None else list(seqs)
    own = cache is None
    cache = cache or make_cache(w, sm_scale=sm_scale, chunk_rows=chunk_rows, fused_merge=fused_merge,
                                policy=policy, keep_first=keep_first, prefill_ws=prefill_ws,
                                chunk_cluster=chunk_cluster, rope_base=rope_base, chunk_barriers=chunk_barriers)
    orc = oracle or OracleCache(len(seqs), w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity,
                                sm_scale=sm_scale, precision="f32", policy=policy, keep_first=keep_first,
                                rope_base=rope_base)
    tol = out_tol(w)
    rep = ParityReport()
    done = 0
    blocks = 0
    while done < n_tokens:
        T = min(block, n_tokens - done)
        p0 = first_pos + done
        if period:
            drawn = [_periodic_token(w, (p0 + t) % period, layer) for t in range(T)]
            q, k, v = (np.stack([d[i] for d in drawn]) for i in range(3))
        else:
            q, k, v = W.tokens(w, p0, T, layer)
        g_out, g_ev = gpu_block(cache, w, q, k, v, p0, use_prefill)
        for t in range(T):
            pos_t = p0 + t
            if direct_fill and orc.len[0] < w.capacity:
                n = int(orc.len[0])
                assert np.all(g_ev[t] == -1)
                orc.K[:, :, n] = k[t][seqs]
                orc.V[:, :, n] = v[t][seqs]
                orc.pos[:, n] = pos_t
                orc.len[:] = n + 1
                continue
            forced = np.full(len(seqs), -1, np.int32)
            full = orc.len[0] == w.capacity
            if full:
                for i, b in enumerate(seqs):
                    e = int(g_ev[t, b])
                    if e == pos_t:
                        forced[i] = w.capacity
                    else:
                        hit = np.nonzero(orc.pos[i] == e)[0]
                        assert hit.size == 1, f"token {pos_t} seq {b}: GPU dropped position {e}, not in the checker's state"
                        forced[i] = int(hit[0])
            o_out, o_ev, victim, argmin, gap, mean = orc.step(q[t][seqs], k[t][seqs], v[t][seqs], pos_t, forced=forced,
                                                              want_mean=full and policy == "tova")
            assert np.all(gap < GAP_TOL), f"token {pos_t}: GPU victim lies {gap.max():.3e} above the minimum"
            if full and policy == "tova":
                for i in np.nonzero(victim != argmin)[0]:
                    low = float(mean[i, argmin[i]])
                    rel = float(gap[i]) / max(low, 1e-30)
                    rep.max_rel_gap = max(rep.max_rel_gap, rel)
                    assert rel <= REL_GAP_TOL, (f"token {pos_t} seq {seqs[i]}: GPU victim's average lies {gap[i]:.3e} "
                                                f"above the lowest ({low:.3e}): more than rounding explains")
            assert np.array_equal(o_ev, g_ev[t, seqs]), f"token {pos_t}: evicted {g_ev[t, seqs]} vs {o_ev}"
            err = float(np.abs(g_out[t][seqs] - o_out).max())
            assert err <= tol, f"token {pos_t}: output error {err:.3e} > {tol}"
            rep.max_err = max(rep.max_err, err)
            rep.max_gap = max(rep.max_gap, float(gap.max()))
            if full:
                rep.evictions += len(seqs)
                rep.resyncs += int(np.sum(victim != argmin))
                rep.self_evictions += int(np.sum(victim == w.capacity))
        rep.evicted_log.append(g_ev)
        done += T
        rep.steps = done
        blocks += 1
        if blocks % check_state_every == 0 or done == n_tokens:
            st = cache.tova_cache_read()
            assert st["status"] == 0, f"device status {st['status']}"
            assert np.array_equal(st["len"].numpy()[seqs], orc.len), "state sizes differ"
            assert np.array_equal(st["positions"].numpy()[seqs], orc.pos), f"slot table differs after {done} tokens"
    rep.cache = cache
    rep.oracle = orc
    return rep


_token_memo = {}


def _periodic_token(w, pos, layer):
    key = (w, pos, layer)
    if key not in _token_memo:
        if len(_token_memo) > 1024:
            _token_memo.clear()
        _token_memo[key] = W.token(w, pos, layer)
    return _token_memo[key]


def run_lockstep_units(w: W.Workload, n_tokens: int, policy: str, recent: int = 0, *, block: int = 64,
                       use_prefill: bool = True, chunk_rows: int = 0, fused_merge: bool = True,
                       score_rtol: float = 1e-5) -> ParityReport:
    """run_lockstep for the policies whose rows are owned per unit (TOVA-head, H2O): dropped positions and slot
    tables per unit bit-exact under the same victim rule (gap measured in the quantity the policy minimises),
    outputs within tolerance, and for H2O the accumulated scores of all slots at the end within score_rtol of their
    size (a sink row's score grows by about half a unit per step: hundreds of fp32 additions on either side)."""
    from oracle.tova_oracle import OracleUnitsCache
    cache = make_cache(w, chunk_rows=chunk_rows, fused_merge=fused_merge, policy=policy, keep_first=recent)
    orc = OracleUnitsCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, policy, recent=recent,
                           precision="f32")
    U = orc.U
    assert cache.tova_cache_units() == U
    tol = out_tol(w)
    rep = ParityReport()
    done = 0
    while done < n_tokens:
        T = min(block, n_tokens - done)
        q, k, v = W.tokens(w, done, T)
        dq, dk, dv = (tova.to_device(a, w.dtype) for a in (q, k, v))
        out = torch.empty(T, w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda:0")
        ev = torch.full((T, w.batch, U), -12345, dtype=torch.int32, device="cuda:0")
        if use_prefill:
            cache.tova_prefill(dq, dk, dv, T, done, out, ev)
        else:
            for t in range(T):
                cache.tova_decode_step(dq[t], dk[t], dv[t], done + t, out[t], ev[t])
        torch.cuda.synchronize()
        g_out, g_ev = out.cpu().numpy(), ev.cpu().numpy()
        for t in range(T):
            pos_t = done + t
            full = orc.len[0] == w.capacity
            forced = np.full((w.batch, U), -1, np.int32)
            if full:
                for b in range(w.batch):
                    for u in range(U):
                        e = int(g_ev[t, b, u])
                        if e == pos_t:
                            forced[b, u] = w.capacity
                        else:
                            hit = np.nonzero(orc.pos[b, u] == e)[0]
                            assert hit.size == 1, f"token {pos_t} seq {b} unit {u}: GPU dropped {e}, not held by the checker"
                            forced[b, u] = int(hit[0])
            o_out, o_ev, victim, argmin, gap, _ = orc.step(q[t], k[t], v[t], pos_t, forced=forced)
            assert np.all(gap < GAP_TOL), f"token {pos_t}: GPU victim lies {gap.max():.3e} above the minimum"
            assert np.array_equal(o_ev, g_ev[t]), f"token {pos_t}: dropped {g_ev[t].tolist()} vs {o_ev.tolist()}"
            err = float(np.abs(g_out[t] - o_out).max())
            assert err <= tol, f"token {pos_t}: output error {err:.3e} > {tol}"
            rep.max_err = max(rep.max_err, err)
            if full:
                rep.evictions += w.batch * U
                rep.resyncs += int(np.sum(victim != argmin))
                rep.self_evictions += int(np.sum(victim == w.capacity))
        done += T
        rep.steps = done
        st = cache.tova_cache_read()
        assert st["status"] == 0
        assert np.array_equal(st["len"].numpy(), orc.len)
        assert np.array_equal(st["positions"].numpy().reshape(w.batch, U, w.capacity), orc.pos), f"slot tables differ after {done} tokens"
    if policy.startswith("h2o"):
        sc = cache.tova_cache_read_scores().numpy()
        assert np.all(np.abs(sc - orc.acc) <= score_rtol * np.maximum(1.0, np.abs(orc.acc))), float(np.abs(sc - orc.acc).max())
    rep.cache, rep.oracle = cache, orc
    return rep


def replay_slot_table(evicted: np.ndarray, capacity: int, first_pos: int = 0) -> np.ndarray:
    """Integer replay of a position log [T,B]: which positions must be held
    after T tokens, as sets per sequence (slot order is not recoverable from
    the log alone)."""
    T, B = evicted.shape
    held = [set() for _ in range(B)]
    for t in range(T):
        for b in range(B):
            held[b].add(first_pos + t)
            e = int(evicted[t, b])
            if e >= 0:
                assert e in held[b], (t, b, e)
                held[b].remove(e)
            assert len(held[b]) <= capacity
    return held
