"""A layer sharded by KV head, on ONE GPU: the ranks are emulated as caches of one process, each holding its share
of the heads, stepping in rank order on one stream (first every rank's scores call, then every rank's commit call,
so no kernel ever waits for one that has not run).  The score tables and flags that would be peer memory are plain
device tensors here.  Held against the checker of the WHOLE layer: outputs of every head, dropped positions,
slot tables - and all ranks must agree with each other."""
import numpy as np
import pytest
import torch

import paper_2401_06104_b200 as tova
from paper_2401_06104_b200 import workloads as W
from oracle.tova_oracle import OracleCache
from parity import GAP_TOL, out_tol

pytestmark = pytest.mark.gpu

MISTRAL = W.WORKLOADS["mistral_7b_gqa"]
LLAMA = W.WORKLOADS["llama2_7b_layer"]


def run_sharded(w, world, n_tokens, mode, keep_first=0, chunk_rows=0, fused=True):
    dev = "cuda:0"
    B, H, Hkv, D, cap = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity
    Hl, Kl = H // world, Hkv // world
    caches = []
    for r in range(world):
        c = tova.TovaCache(B, Hl, Kl, D, cap, dtype=w.dtype)
        if chunk_rows:
            c.tova_cache_set_chunk_rows(chunk_rows)
        if not fused:
            c.tova_cache_set_fused_merge(False)
        if keep_first:
            c.tova_cache_set_policy(tova.TOVA_POLICY_TOVA, keep_first)
        caches.append(c)
    ld = (cap + 1 + 3) // 4 * 4
    if mode == "peer":
        nb = caches[0].tova_shard_table_bytes(world)
        assert nb == 2 * world * B * ld * 4
        tables = [torch.zeros(nb // 4, dtype=torch.float32, device=dev) for _ in range(world)]
        flags = [torch.zeros(world, dtype=torch.int32, device=dev) for _ in range(world)]
        for r, c in enumerate(caches):
            c.tova_cache_set_shard(r, world, H, tables, flags)
    else:
        tables = [torch.zeros(B, ld, dtype=torch.float32, device=dev) for _ in range(world)]
        for r, c in enumerate(caches):
            c.tova_cache_set_shard(r, world, H, [tables[i] if i == r else None for i in range(world)], None)
    orc = OracleCache(B, H, Hkv, D, cap, precision="f32", keep_first=keep_first)
    outs = [torch.empty(B, Hl, D, device=dev) for _ in range(world)]
    evs = [torch.full((B,), -9, dtype=torch.int32, device=dev) for _ in range(world)]
    worst, resyncs = 0.0, 0
    for t in range(n_tokens):
        q, k, v = W.token(w, t)
        parts = []
        for r in range(world):
            parts.append(tuple(tova.to_device(np.ascontiguousarray(a), w.dtype) for a in
                               (q[:, r * Hl:(r + 1) * Hl], k[:, r * Kl:(r + 1) * Kl], v[:, r * Kl:(r + 1) * Kl])))
        full = caches[0].tova_cache_len() == cap
        for r, c in enumerate(caches):
            c.tova_decode_step_scores(*parts[r], t, outs[r])
        if mode == "reduce" and full:                  # what an all-reduce would leave on every rank
            total = torch.stack(tables).sum(dim=0)
            for tb in tables:
                tb.copy_(total)
        for r, c in enumerate(caches):
            c.tova_decode_step_commit(parts[r][1], parts[r][2], evs[r])
        torch.cuda.synchronize()
        ev = evs[0].cpu().numpy()
        for r in range(1, world):
            assert np.array_equal(evs[r].cpu().numpy(), ev), f"token {t}: ranks disagree about the victim"
        forced = np.full(B, -1, np.int32)
        if full:
            for b in range(B):
                e = int(ev[b])
                forced[b] = cap if e == t else int(np.nonzero(orc.pos[b] == e)[0][0])
        o_out, o_ev, victim, argmin, gap, _ = orc.step(q, k, v, t, forced=forced)
        assert np.all(gap < GAP_TOL), (t, gap)
        assert np.array_equal(o_ev, ev), (t, o_ev, ev)
        g_out = torch.cat(outs, dim=1).cpu().numpy()
        err = float(np.abs(g_out - o_out).max())
        assert err <= out_tol(w), (t, err)
        worst = max(worst, err)
        resyncs += int(np.sum(victim != argmin))
    for r, c in enumerate(caches):
        st = c.tova_cache_read(want_kv=True)
        assert st["status"] == 0
        assert np.array_equal(st["positions"].numpy(), orc.pos)
        assert np.array_equal(st["K"].numpy(), orc.K[:, r * Kl:(r + 1) * Kl])
        assert np.array_equal(st["V"].numpy(), orc.V[:, r * Kl:(r + 1) * Kl])
    return worst, resyncs


@pytest.mark.parametrize("mode", ["peer", "reduce"])
@pytest.mark.parametrize("world,H,Hkv", [(2, 8, 4), (4, 8, 4), (2, 16, 2), (8, 8, 8)])
def test_sharded_layer_matches_the_checker_of_the_whole_layer(world, H, Hkv, mode):
    w = MISTRAL.scaled(batch=2, n_q_heads=H, n_kv_heads=Hkv, capacity=90)
    run_sharded(w, world, 90 + 120, mode)


def test_sharded_layer_with_protected_positions_and_the_global_memory_merge():
    w = LLAMA.scaled(batch=2, n_q_heads=8, n_kv_heads=8, capacity=300)
    run_sharded(w, 2, 300 + 40, "peer", keep_first=3, chunk_rows=32, fused=False)


def test_sharded_step_call_order_and_refusals():
    w = MISTRAL.scaled(batch=1, n_q_heads=4, n_kv_heads=2, capacity=8)
    c = tova.TovaCache(1, 2, 1, 128, 8, dtype=w.dtype)
    tab = torch.zeros(1, 12, dtype=torch.float32, device="cuda:0")
    q = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda:0")
    k = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros(1, 2, 128, device="cuda:0")
    with pytest.raises(tova.TovaError):
        c.tova_decode_step_scores(q, k, k, 0, out)              # not a sharded cache
    with pytest.raises(tova.TovaError):
        c.tova_cache_set_shard(2, 2, 4, [tab, tab], None)       # rank out of range
    c.tova_cache_set_shard(1, 2, 4, [None, tab], None)
    with pytest.raises(tova.TovaError):
        c.tova_decode_step(q, k, k, 0, out)                     # the one-call step is refused on a sharded cache
    with pytest.raises(tova.TovaError):
        c.tova_prefill(q[None], k[None], k[None], 1, 0, out[None])   # nor prompts
    with pytest.raises(tova.TovaError):
        c.tova_cache_set_policy(tova.TOVA_POLICY_WINDOW, 0)     # the exchange sums TOVA's weights
    with pytest.raises(tova.TovaError):
        c.tova_decode_step_commit(k, k)                         # nothing scored yet
    c.tova_decode_step_scores(q, k, k, 0, out)
    with pytest.raises(tova.TovaError):
        c.tova_decode_step_scores(q, k, k, 1, out)              # a commit is outstanding
    c.tova_decode_step_commit(k, k)
    assert c.tova_cache_len() == 1


def test_a_rank_that_never_reports_is_detected_without_hanging():
    """World of 2, but only rank 0 exists: its commit waits for rank 1's flag, gives up after its bounded wait and
    leaves a status code; the state is untouched and the context stays usable."""
    w = MISTRAL.scaled(batch=1, n_q_heads=4, n_kv_heads=2, capacity=4)
    c = tova.TovaCache(1, 2, 1, 128, 4, dtype=w.dtype)
    nb = c.tova_shard_table_bytes(2)
    tabs = [torch.zeros(nb // 4, dtype=torch.float32, device="cuda:0") for _ in range(2)]
    flags = [torch.zeros(2, dtype=torch.int32, device="cuda:0") for _ in range(2)]
    c.tova_cache_set_shard(0, 2, 4, tabs, flags)
    out = torch.zeros(1, 2, 128, device="cuda:0")
    ev = torch.full((1,), -9, dtype=torch.int32, device="cuda:0")
    for t in range(5):
        tq, tk, tv = W.token(w, t)
        q, k, v = (tova.to_device(np.ascontiguousarray(a), w.dtype) for a in (tq[:, :2], tk[:, :1], tv[:, :1]))
        c.tova_decode_step_scores(q, k, v, t, out)
        c.tova_decode_step_commit(k, v, ev)
    torch.cuda.synchronize()
    st = c.tova_cache_read()
    assert st["status"] == 3                                     # a peer's part did not arrive
    # the four filling steps reported -1; the step that timed out wrote nothing and changed nothing
    assert st["positions"][0].tolist() == [0, 1, 2, 3] and int(ev.item()) == -1
