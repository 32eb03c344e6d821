"""Parity at the full layer shapes, in the launch configuration the benchmark
times (automatic chunk size, tova_prefill blocks): the checker follows a
sample of the sequences token by token; an integer replay of the eviction log
checks every sequence's slot table."""
import numpy as np
import pytest

from paper_2401_06104_b200 import workloads as W
from parity import make_cache, replay_slot_table, run_lockstep

pytestmark = pytest.mark.gpu


def check_all_sequences(rep, w, n_tokens):
    log = np.concatenate(rep.evicted_log, axis=0)
    held = replay_slot_table(log, w.capacity)
    st = rep.cache.tova_cache_read()
    assert st["status"] == 0
    pos = st["positions"].numpy()
    for b in range(w.batch):
        live = [p for p in pos[b].tolist() if p >= 0]
        assert len(live) == len(set(live)) == min(n_tokens, w.capacity)
        assert set(live) == held[b]


@pytest.mark.parametrize("name,cap,extra,seqs,direct_fill", [
    ("llama2_7b_layer", 512, 160, [0, 5], False),
    ("mistral_7b_gqa", 256, 200, [3], False),
    ("mistral_7b_gqa", 1024, 96, [17], False),
    ("mistral_7b_gqa", 4096, 32, [30], True),
    ("yi_6b_long", 4096, 40, [1], True),
])
def test_full_layer_shapes(name, cap, extra, seqs, direct_fill):
    w = W.WORKLOADS[name].scaled(capacity=cap)
    n = cap + extra
    rep = run_lockstep(w, n, seqs=seqs, block=128, check_state_every=1000, direct_fill=direct_fill)
    assert rep.evictions == len(seqs) * extra
    assert rep.resyncs <= max(1, rep.evictions // 20)      # the two sides may differ on near-ties only: rare
    check_all_sequences(rep, w, n)
    print(f"{name} k={cap}: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions} "
          f"self {rep.self_evictions}")


@pytest.mark.parametrize("name,cap,seqs", [("mistral_7b_gqa", 1024, [5, 31]), ("llama2_7b_layer", 512, [0, 7]),
                                           ("yi_6b_long", 4096, [2])])
def test_chunked_prompt_at_full_layer_shapes(name, cap, seqs):
    """512-token tova_prefill calls onto a full state (eight chunks of 64 each), full batch, the checker on
    sampled sequences, the slot tables of all sequences replayed from the log."""
    w = W.WORKLOADS[name].scaled(capacity=cap)
    n = cap + (512 if cap <= 1024 else 128)
    rep = run_lockstep(w, n, seqs=seqs, block=512 if cap <= 1024 else 128, check_state_every=1000, direct_fill=True,
                       prefill_ws=True)
    assert rep.evictions == len(seqs) * (n - cap)
    assert rep.resyncs <= max(1, rep.evictions // 20)
    check_all_sequences(rep, w, n)
    print(f"{name} k={cap} chunked prompt: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions}")


def test_position_compression_at_the_layer_shape():
    """B=8, 32 MHA heads, state of 512 rows, q and k without rotary embedding: the rotating streaming kernel at
    the shape the paper's extrapolation experiment uses (multi-state 512), the checker on two sequences."""
    w = W.WORKLOADS["llama2_7b_layer"].scaled(rope=False)
    n = w.capacity + 96
    rep = run_lockstep(w, n, seqs=[0, 6], block=128, check_state_every=1000, direct_fill=True, rope_base=10000.0)
    assert rep.evictions == 2 * 96 and rep.resyncs <= 9
    check_all_sequences(rep, w, n)
    print(f"position compression k=512 B=8: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions}")


def test_per_head_policy_at_the_full_gqa_shape():
    """TOVA-head on the Mistral shape (B=32, 32 query / 8 KV heads, state of 1024 rows): while the state fills no
    head drops anything, so the checker's per-head tables are written directly; then 40 tokens in lock step on two
    sequences, every KV head dropping its own row."""
    import torch
    import paper_2401_06104_b200 as tova
    from oracle.tova_oracle import OracleUnitsCache
    from parity import GAP_TOL, out_tol
    w = W.WORKLOADS["mistral_7b_gqa"].scaled(capacity=1024)
    seqs, extra = [4, 27], 40
    cache = make_cache(w, policy="tova_head")
    U = w.n_kv_heads
    orc = OracleUnitsCache(len(seqs), w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, "tova_head", precision="f32")
    done = 0
    while done < w.capacity + extra:
        T = min(128, w.capacity + extra - done)
        q, k, v = W.tokens(w, done, T)
        dq, dk, dv = (tova.to_device(a, w.dtype) for a in (q, k, v))
        out = torch.empty(T, w.batch, w.n_q_heads, w.head_dim, device="cuda:0")
        ev = torch.empty(T, w.batch, U, dtype=torch.int32, device="cuda:0")
        cache.tova_prefill(dq, dk, dv, T, done, out, ev)
        torch.cuda.synchronize()
        g_out, g_ev = out.cpu().numpy(), ev.cpu().numpy()
        for t in range(T):
            pos_t = done + t
            if orc.len[0] < w.capacity:
                n = int(orc.len[0])
                assert np.all(g_ev[t] == -1)
                orc.K[:, :, n], orc.V[:, :, n] = k[t][seqs], v[t][seqs]
                orc.pos[:, :, n] = pos_t
                orc.len[:] = n + 1
                continue
            forced = np.zeros((len(seqs), U), np.int32)
            for i, b in enumerate(seqs):
                for u in range(U):
                    e = int(g_ev[t, b, u])
                    forced[i, u] = w.capacity if e == pos_t else int(np.nonzero(orc.pos[i, u] == e)[0][0])
            o_out, o_ev, victim, argmin, gap, _ = orc.step(q[t][seqs], k[t][seqs], v[t][seqs], pos_t, forced=forced)
            assert np.all(gap < GAP_TOL) and np.array_equal(o_ev, g_ev[t, seqs]), pos_t
            assert np.abs(g_out[t][seqs] - o_out).max() <= out_tol(w), pos_t
            assert np.sum(victim != argmin) == 0
        done += T
    st = cache.tova_cache_read()
    assert st["status"] == 0
    pos = st["positions"].numpy()
    assert np.array_equal(pos[seqs], orc.pos)
    assert any(set(pos[seqs[0], 0].tolist()) != set(pos[seqs[0], u].tolist()) for u in range(1, U))   # heads diverged


def test_sharded_layer_at_a_long_state():
    """Four emulated ranks, two KV heads each, state of 1024 rows (8 chunks per head: the in-kernel merge), batch 4."""
    from test_gpu_sharded import run_sharded
    w = W.WORKLOADS["mistral_7b_gqa"].scaled(batch=4, capacity=1024)
    worst, resyncs = run_sharded(w, 4, 1024 + 24, "peer")
    assert resyncs <= 2
    print(f"sharded mistral k=1024 B=4 world=4: max_err {worst:.2e} resyncs {resyncs}")


def test_32_layer_configuration_at_full_batch():
    """Batch 64, 32 MHA heads, state of 1024 rows: 2048 eight-warp thread blocks of 128-row chunks per streaming
    launch (the launch the benchmark's headline times).  The checker follows three of the 64 sequences."""
    w = W.WORKLOADS["llama2_7b_full"]
    extra = 64
    rep = run_lockstep(w, w.capacity + extra, seqs=[0, 29, 63], block=128, check_state_every=1000, direct_fill=True)
    assert rep.evictions == 3 * extra
    assert rep.resyncs <= max(1, rep.evictions // 20)
    check_all_sequences(rep, w, w.capacity + extra)
    print(f"llama2_7b_full k=1024 B=64: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions} "
          f"max_rel_gap {rep.max_rel_gap:.2e} self {rep.self_evictions}")


def test_unbounded_arm_state_of_8192_rows_at_full_batch():
    """The 8192-token context held whole at batch 64: 64 chunks per head, more than a cluster merges, so every
    streaming warp is its own thread block and the partials go through global memory (131072 blocks per launch).
    The state fills without any deletion; the last steps run on the full state and drop rows.  Tokens repeat with
    period 512 (see run_lockstep), so the lowest average is shared by 16 rows and the lowest slot must win."""
    w = W.WORKLOADS["llama2_7b_full"].scaled(capacity=8192)
    extra = 6
    rep = run_lockstep(w, w.capacity + extra, seqs=[1, 62], block=128, check_state_every=1000, direct_fill=True,
                       period=512)
    assert rep.evictions == 2 * extra
    check_all_sequences(rep, w, w.capacity + extra)
    print(f"llama2_7b_full k=8192 B=64: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions} "
          f"max_rel_gap {rep.max_rel_gap:.2e}")


def test_long_stream_of_70000_tokens():
    """The whole long-stream configuration on the GPU: 4096 prompt tokens and 65,904 decode tokens through a state
    of 4096 rows, all four sequences.  The checker cannot follow 70,000 tokens (minutes per thousand at this
    size), so it joins at checkpoints: there its state is written from the GENERATOR's tokens at the positions the
    GPU's slot table holds (after checking that the GPU's cached rows are bit for bit those tokens), and the next 32
    tokens are compared token by token - dropped positions exact, outputs within tolerance.  Over the whole stream
    an integer replay of the dropped-position log must reproduce the final slot table, and no kernel may have
    reported a failed check."""
    import torch
    import paper_2401_06104_b200 as tova
    from oracle.tova_oracle import OracleCache
    w = W.WORKLOADS["yi_6b_long"]
    total = w.prompt + w.decode
    assert total == 70000 and w.capacity == 4096
    cache = make_cache(w)
    checkpoints = [4096, 4128, 9001, 20000, 33333, 47111, 61000, total - 32]
    span = 32
    logs = []
    pos = 0
    worst, resyncs, evictions = 0.0, 0, 0
    for cp in checkpoints:
        while pos < cp:                                   # plain GPU run up to the checkpoint
            T = min(1024, cp - pos)
            q, k, v = W.tokens(w, pos, T)
            dq, dk, dv = (tova.to_device(a, w.dtype) for a in (q, k, v))
            ev = torch.empty(T, w.batch, dtype=torch.int32, device="cuda:0")
            cache.tova_prefill(dq, dk, dv, T, pos, None, ev)
            torch.cuda.synchronize()
            logs.append(ev.cpu().numpy())
            pos += T
        st = cache.tova_cache_read(want_kv=True)
        assert st["status"] == 0 and np.all(st["len"].numpy() == w.capacity)
        held = st["positions"].numpy()
        orc = OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, precision="f32")
        for p_held in np.unique(held):
            _, k1, v1 = W.token(w, int(p_held))
            for b, s in zip(*np.nonzero(held == p_held)):
                orc.K[b, :, s] = k1[b]
                orc.V[b, :, s] = v1[b]
        assert np.array_equal(st["K"].numpy(), orc.K) and np.array_equal(st["V"].numpy(), orc.V), cp
        orc.pos[:] = held
        orc.len[:] = w.capacity
        rep = run_lockstep(w, span, cache=cache, oracle=orc, first_pos=pos, block=span)
        logs.extend(rep.evicted_log)
        pos += span
        worst = max(worst, rep.max_err)
        resyncs += rep.resyncs
        evictions += rep.evictions
    assert pos == total
    log = np.concatenate(logs, axis=0)
    assert log.shape == (total, w.batch)
    held = replay_slot_table(log, w.capacity)
    st = cache.tova_cache_read()
    assert st["status"] == 0
    for b in range(w.batch):
        live = st["positions"].numpy()[b].tolist()
        assert len(set(live)) == w.capacity and set(live) == held[b]
        assert 0 in held[b]                               # the sink (position 0) is still held, as in Section 7.3
    assert evictions == w.batch * span * len(checkpoints) and resyncs <= evictions // 20
    print(f"yi_6b_long 70000 tokens: max_err {worst:.2e} resyncs {resyncs}/{evictions}")


@pytest.mark.parametrize("name,cap", [("llama2_7b_layer", 512), ("mistral_7b_gqa", 1024), ("yi_6b_long", 4096)])
def test_full_shapes_as_the_benchmark_launches_them(name, cap):
    """Deferred eviction, two layer caches taking turns, steps replayed from a CUDA
    graph with positions from the device counter: bit-identical outputs, dropped
    positions and state to plain stream-ordered steps (which the test above holds
    against the checker)."""
    import torch
    import paper_2401_06104_b200 as tova
    w = W.WORKLOADS[name].scaled(capacity=cap)
    L, G, R = 2, 8, 3                      # caches, steps per graph, replays
    n_fill = cap + 8
    toks = [W.tokens(w, 0, n_fill + G * R, layer=l) for l in range(L)]
    dev = [[tova.to_device(a, w.dtype) for a in t] for t in toks]
    ref = [make_cache(w) for _ in range(L)]
    dfr = [make_cache(w) for _ in range(L)]
    for l in range(L):
        for c in (ref[l], dfr[l]):
            c.tova_prefill(dev[l][0], dev[l][1], dev[l][2], n_fill, 0, None, None)
    shape = (G * R, w.batch, w.n_q_heads, w.head_dim)
    o_ref = [torch.empty(shape, device="cuda:0") for _ in range(L)]
    e_ref = [torch.full((G * R, w.batch), -7, dtype=torch.int32, device="cuda:0") for _ in range(L)]
    for t in range(G * R):
        for l in range(L):
            q, k, v = (a[n_fill + t] for a in dev[l])
            ref[l].tova_decode_step(q, k, v, n_fill + t, o_ref[l][t], e_ref[l][t])
    # the benchmark's way: static input/output buffers, one graph of G steps per cache, replayed
    for c in dfr:
        c.tova_cache_set_deferred_eviction(True)
    sq = [[torch.empty_like(a[:G]) for a in dev[l]] for l in range(L)]
    so = [torch.empty((G,) + shape[1:], device="cuda:0") for _ in range(L)]
    se = [torch.full((G, w.batch), -7, dtype=torch.int32, device="cuda:0") for _ in range(L)]
    o_dfr = [torch.empty(shape, device="cuda:0") for _ in range(L)]
    e_dfr = [torch.empty((G * R, w.batch), dtype=torch.int32, device="cuda:0") for _ in range(L)]

    def steps():
        for t in range(G):
            for l in range(L):
                dfr[l].tova_decode_step(sq[l][0][t], sq[l][1][t], sq[l][2][t], -1, so[l][t], se[l][t])
        for c in dfr:
            c.tova_cache_join()

    def load(r):
        for l in range(L):
            for i in range(3):
                sq[l][i].copy_(dev[l][i][n_fill + r * G: n_fill + (r + 1) * G])

    side = torch.cuda.Stream()
    load(0)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        steps()                              # replay 0 runs directly (sets function attributes before capture)
        side.synchronize()
        for l in range(L):
            o_dfr[l][:G].copy_(so[l]); e_dfr[l][:G].copy_(se[l])
        load(1)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            steps()
    for r in range(1, R):
        if r > 1:
            load(r)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        for l in range(L):
            o_dfr[l][r * G:(r + 1) * G].copy_(so[l]); e_dfr[l][r * G:(r + 1) * G].copy_(se[l])
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(e_ref[l], e_dfr[l]), f"{name} layer {l}: dropped positions differ"
        assert torch.equal(o_ref[l], o_dfr[l]), f"{name} layer {l}: outputs differ"
        a, b = ref[l].tova_cache_read(), dfr[l].tova_cache_read()
        assert a["status"] == 0 and b["status"] == 0
        assert torch.equal(a["positions"], b["positions"]) and torch.equal(a["len"], b["len"])


@pytest.mark.parametrize("mode", [1, 2])   # 1: tcgen05 kernel; 2: warp-level MMA kernel
@pytest.mark.parametrize("name,cap", [("llama2_7b_layer", 512), ("mistral_7b_gqa", 1024), ("yi_6b_long", 4096)])
def test_bulk_prefill_full_shapes_on_sampled_tokens(name, cap, mode):
    """A prompt that fills the whole state in one tova_prefill call (one bulk run: rows copied, one causal-attention
    launch, one commit).  The state must be the prompt in order; the outputs of sampled (token, sequence) pairs are
    recomputed by the checker, whose state is written with the tokens before the sampled one."""
    from oracle.tova_oracle import OracleCache
    from parity import gpu_block, out_tol
    w = W.WORKLOADS[name].scaled(capacity=cap)
    T = cap
    q, k, v = W.tokens(w, 0, T)
    cache = make_cache(w)
    cache.tova_cache_set_bulk_prefill(mode)
    out, ev = gpu_block(cache, w, q, k, v, 0)
    assert cache.tova_cache_launches() == 1 + 3
    assert np.all(ev == -1)
    st = cache.tova_cache_read(want_kv=True)
    assert st["status"] == 0
    assert np.all(st["len"].numpy() == cap)
    assert np.array_equal(st["positions"].numpy(), np.tile(np.arange(cap, dtype=np.int32), (w.batch, 1)))
    assert np.array_equal(st["K"].float().numpy(), k.transpose(1, 2, 0, 3))
    assert np.array_equal(st["V"].float().numpy(), v.transpose(1, 2, 0, 3))
    worst = 0.0
    for b in sorted({0, w.batch // 2, w.batch - 1}):
        for t in sorted({0, 1, 15, 16, 63, 64, 65, 127, 128, cap // 2 - 1, cap // 2 + 37, cap - 65, cap - 2, cap - 1}):
            orc = OracleCache(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, precision="f32")
            orc.K[0, :, :t] = k[:t, b].transpose(1, 0, 2)
            orc.V[0, :, :t] = v[:t, b].transpose(1, 0, 2)
            orc.pos[0, :t] = np.arange(t)
            orc.len[:] = t
            o, e, *_ = orc.step(q[t, b:b + 1], k[t, b:b + 1], v[t, b:b + 1], t)
            assert e[0] == -1
            err = float(np.abs(o[0] - out[t, b]).max())
            assert err <= out_tol(w), (b, t, err)
            worst = max(worst, err)
    print(f"{name} k={cap}: bulk prefill max_err {worst:.2e}")
