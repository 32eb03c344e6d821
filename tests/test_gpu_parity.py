"""GPU parity: the CUDA library, called through the C ABI, against the CPU
checker on the same seeded inputs.  Retained positions are compared slot by
slot (bit-exact), outputs within 2e-3 (bf16 inputs) / 1e-5 (fp32 inputs)."""
import os

import numpy as np
import pytest
import torch

import paper_2401_06104_b200 as tova
from paper_2401_06104_b200 import workloads as W
from oracle.tova_oracle import OracleCache
from parity import gpu_block, hand_tol, make_cache, out_tol, replay_slot_table, run_lockstep, run_lockstep_units
from test_oracle_pins import parse_golden

pytestmark = pytest.mark.gpu

LLAMA = W.WORKLOADS["llama2_7b_layer"]
MISTRAL = W.WORKLOADS["mistral_7b_gqa"]
YI = W.WORKLOADS["yi_6b_long"]


def test_hand_worked_example_on_gpu():
    """The 3-row example (exact tie, self-eviction, slot order != position order)."""
    toks, steps = parse_golden()
    D = 64
    c = tova.TovaCache(1, 2, 2, D, 3, dtype=tova.TOVA_DTYPE_FP32, sm_scale=1.0)
    out = torch.empty(1, 2, D, device="cuda:0")
    ev = torch.empty(1, dtype=torch.int32, device="cuda:0")
    for (t, e, rows_after, o0, o1) in steps:
        q = np.zeros((1, 2, D), np.float32); q[..., 0] = 1.0
        k = np.zeros((1, 2, D), np.float32); v = np.zeros((1, 2, D), np.float32)
        a0, v0, a1, v1 = toks[t]
        k[0, 0, 0], k[0, 1, 0] = np.log(a0), np.log(a1)
        v[0, 0, 0], v[0, 1, 0] = v0, v1
        c.tova_decode_step(*(tova.to_device(a, 0) for a in (q, k, v)), t, out, ev)
        st = c.tova_cache_read()
        assert int(ev.item()) == e, t
        assert st["positions"][0].tolist() == rows_after, t
        o = out.cpu().numpy()
        assert abs(o[0, 0, 0] - float(o0)) <= hand_tol(float(o0)) and abs(o[0, 1, 0] - float(o1)) <= hand_tol(float(o1))
        assert np.all(o[0, :, 1:] == 0)
        assert st["status"] == 0 and c.tova_cache_len() == min(t + 1, 3)


@pytest.mark.parametrize("name", ["tiny", "tiny_unit"])
def test_tiny_reference_config_full_stream(name):
    """1 layer, batch 1, 4 MHA heads, D 64, fp32, capacity 64, 32 + 512 tokens."""
    w = W.WORKLOADS[name]
    rep = run_lockstep(w, w.prompt + w.decode, block=32)
    assert rep.evictions == w.prompt + w.decode - w.capacity
    print(f"{name}: resyncs {rep.resyncs}/{rep.evictions} self {rep.self_evictions} "
          f"max_err {rep.max_err:.2e} max_gap {rep.max_gap:.2e}")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("chunk_rows", [0, 32, 64, 96, 128, 256, 1024])
def test_llama_shape_reduced_every_chunk_size(chunk_rows, fused):
    """bf16 MHA, capacity 203: several tiles plus a ragged tail at every chunk
    size, with the partials merged inside the streaming kernel (clusters of 1 to
    7 warps) and through global memory."""
    w = LLAMA.scaled(batch=2, n_q_heads=6, n_kv_heads=6, capacity=203)
    rep = run_lockstep(w, 460, chunk_rows=chunk_rows, block=50, fused_merge=fused)
    assert rep.evictions == 2 * (460 - 203)


@pytest.mark.parametrize("H,Hkv", [(6, 6), (8, 2), (16, 1)])
def test_head_groups_spanning_several_ctas(H, Hkv):
    """Capacity 300 in 32-row chunks: 10 chunks, i.e. two CTAs of 5 warps per head
    group that merge across a cluster (1 to 2 CTAs while the state fills); and 8
    chunks exactly (capacity 256), the largest single CTA."""
    w = LLAMA.scaled(batch=2, n_q_heads=H, n_kv_heads=Hkv, capacity=300)
    rep = run_lockstep(w, 300 + 120, chunk_rows=32, block=60)
    assert rep.evictions == 2 * 120
    w = LLAMA.scaled(batch=2, n_q_heads=H, n_kv_heads=Hkv, capacity=256)
    rep = run_lockstep(w, 256 + 100, chunk_rows=32, block=60)
    assert rep.evictions == 2 * 100


@pytest.mark.parametrize("H,Hkv,cap", [(4, 4, 2040), (8, 2, 1500), (2, 2, 2100)])
def test_cluster_sizes_up_to_eight_and_beyond(H, Hkv, cap):
    """32-row chunks: 64 chunks (8 CTAs x 8 warps, the largest cluster), 47 chunks
    (6 CTAs, ragged), and 66 chunks, which no cluster holds: partials through
    global memory although the fused merge is on."""
    w = LLAMA.scaled(batch=1, n_q_heads=H, n_kv_heads=Hkv, capacity=cap)
    rep = run_lockstep(w, cap + 40, chunk_rows=32, block=64, direct_fill=True, check_state_every=8)
    assert rep.evictions == 40


@pytest.mark.parametrize("H,Hkv,D,dtype,cap,B", [
    (8, 2, 128, W.DTYPE_BF16, 200, 3),      # G = 4 (Mistral-like)
    (16, 2, 128, W.DTYPE_BF16, 130, 2),     # G = 8 (Yi-like)
    (6, 2, 128, W.DTYPE_BF16, 77, 2),       # G = 3: group not a multiple of the head block
    (32, 2, 64, W.DTYPE_BF16, 65, 1),       # G = 16, D = 64
    (4, 2, 64, W.DTYPE_BF16, 64, 2),        # G = 2, D = 64
    (4, 4, 128, W.DTYPE_FP32, 97, 2),       # fp32, D = 128
    (8, 2, 64, W.DTYPE_FP32, 40, 2),        # fp32 GQA, D = 64
    (2, 1, 128, W.DTYPE_BF16, 1, 2),        # capacity 1: every step evicts
    (4, 4, 128, W.DTYPE_BF16, 33, 1),       # one row past a tile
])
@pytest.mark.parametrize("fused", [True, False])
def test_head_layouts_and_dtypes(H, Hkv, D, dtype, cap, B, fused):
    w = MISTRAL.scaled(batch=B, n_q_heads=H, n_kv_heads=Hkv, head_dim=D, dtype=dtype, capacity=cap)
    rep = run_lockstep(w, cap + 150, block=40, fused_merge=fused)
    assert rep.evictions == B * 150


def test_yi_shape_reduced_with_periodic_heavy_keys():
    w = YI.scaled(batch=2, capacity=256, heavy_period=64)
    rep = run_lockstep(w, 256 + 300, block=64)
    assert rep.evictions == 2 * 300


def test_prefill_equals_decode_steps_bitwise():
    """Per-token route of tova_prefill (bulk processing off): the same launches as decode steps."""
    w = LLAMA.scaled(batch=2, n_q_heads=8, n_kv_heads=8, capacity=100)
    T = 260
    q, k, v = W.tokens(w, 0, T)
    a, b = make_cache(w), make_cache(w)
    a.tova_cache_set_bulk_prefill(False)
    oa, ea = gpu_block(a, w, q, k, v, 0, use_prefill=True)
    ob, eb = gpu_block(b, w, q, k, v, 0, use_prefill=False)
    assert np.array_equal(oa, ob) and np.array_equal(ea, eb)
    sa, sb = a.tova_cache_read(want_kv=True), b.tova_cache_read(want_kv=True)
    for key in ("len", "positions", "K", "V"):
        assert torch.equal(sa[key], sb[key]), key
    assert a.tova_cache_launches() == b.tova_cache_launches() == 1 + 2 * T


@pytest.mark.parametrize("H,Hkv,D,cap,T0,T1", [
    (8, 8, 128, 300, 200, 330),    # MHA; 4 query tiles with a ragged tail, then a run onto 200 held rows, then full
    (8, 2, 128, 130, 7, 200),      # GQA; a short run first (one ragged tile), second run crosses tile borders
    (4, 4, 64, 96, 96, 40),        # D = 64; the run fills the state exactly
    (16, 1, 128, 257, 3, 254),     # below the bulk threshold first (per-token), then a run from 3 held rows
])
@pytest.mark.parametrize("mode", [1, 2])   # 1: tcgen05 kernel where D = 128; 2: warp-level MMA kernel
def test_bulk_prefill_against_decode_steps(H, Hkv, D, cap, T0, T1, mode):
    """The bulk route for tokens that fill free rows: state, dropped positions and all later outputs bit-identical
    to decode steps; outputs of the bulk tokens within the output tolerance (other summation order)."""
    w = LLAMA.scaled(batch=3, n_q_heads=H, n_kv_heads=Hkv, head_dim=D, capacity=cap)
    T = T0 + T1
    q, k, v = W.tokens(w, 0, T)
    a, b = make_cache(w), make_cache(w)
    a.tova_cache_set_bulk_prefill(mode)
    o0, e0 = gpu_block(a, w, q[:T0], k[:T0], v[:T0], 0, use_prefill=True)
    o1, e1 = gpu_block(a, w, q[T0:], k[T0:], v[T0:], T0, use_prefill=True)
    oa, ea = np.concatenate([o0, o1]), np.concatenate([e0, e1])
    ob, eb = gpu_block(b, w, q, k, v, 0, use_prefill=False)
    assert np.array_equal(ea, eb)
    fill = min(T, cap)
    assert np.all(ea[:fill] == -1)
    assert np.abs(oa[:fill] - ob[:fill]).max() <= out_tol(w)
    assert np.array_equal(oa[fill:], ob[fill:])
    sa, sb = a.tova_cache_read(want_kv=True), b.tova_cache_read(want_kv=True)
    assert sa["status"] == 0
    for key in ("len", "positions", "K", "V"):
        assert torch.equal(sa[key], sb[key]), key
    assert a.tova_cache_launches() < b.tova_cache_launches()


def test_bulk_prefill_head_wise_tova_against_decode_steps():
    """Head-wise TOVA: the prompt tokens that find free rows take the bulk route too (every KV head's slot table
    gets the same positions, nothing is dropped); per-unit dropped positions, slot tables, rows and all later outputs
    bit-identical to decode steps, outputs of the bulk tokens within the output tolerance."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=4, capacity=150)
    T0, T1 = 90, 140
    T, U = T0 + T1, w.n_kv_heads
    q, k, v = W.tokens(w, 0, T)
    dq, dk, dv = (tova.to_device(x, w.dtype) for x in (q, k, v))
    caches, outs, evs = [], [], []
    for bulk in (True, False):
        c = make_cache(w)
        c.tova_cache_set_policy(tova.TOVA_POLICY_TOVA_HEAD, 0)
        out = torch.empty(T, w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32, device="cuda:0")
        ev = torch.full((T, w.batch, U), -12345, dtype=torch.int32, device="cuda:0")
        if bulk:
            c.tova_prefill(dq[:T0], dk[:T0], dv[:T0], T0, 0, out[:T0], ev[:T0])
            c.tova_prefill(dq[T0:], dk[T0:], dv[T0:], T1, T0, out[T0:], ev[T0:])
        else:
            for t in range(T):
                c.tova_decode_step(dq[t], dk[t], dv[t], t, out[t], ev[t])
        torch.cuda.synchronize()
        caches.append(c); outs.append(out.cpu().numpy()); evs.append(ev.cpu().numpy())
    assert np.array_equal(evs[0], evs[1])
    assert np.all(evs[0][:w.capacity] == -1) and np.any(evs[0][w.capacity:] >= 0)
    assert np.abs(outs[0][:w.capacity] - outs[1][:w.capacity]).max() <= out_tol(w)
    assert np.array_equal(outs[0][w.capacity:], outs[1][w.capacity:])
    sa, sb = (c.tova_cache_read(want_kv=True) for c in caches)
    assert sa["status"] == 0 and sb["status"] == 0
    for key in ("len", "positions", "K", "V"):
        assert torch.equal(sa[key], sb[key]), key
    assert caches[0].tova_cache_launches() < caches[1].tova_cache_launches()


# ---------------------------------------------------------------------------
# prompt tokens that meet a full state, in chunks (appendix "Experimental Details": whole chunks at once,
# the attention masked according to the layer's attention weights)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("H,Hkv,D,cap,B,block,keep", [
    (8, 8, 128, 203, 2, 64, 0),      # MHA, odd capacity (the chunk's logit columns start at an odd index), whole chunks
    (8, 2, 128, 256, 3, 50, 0),      # GQA, ragged chunks of 50
    (16, 1, 128, 130, 2, 200, 0),    # 200-token calls: three chunks of 64, then 8 tokens as a short chunk
    (4, 4, 64, 96, 2, 71, 0),        # D = 64; 64 + 7: the 7 left over go token by token
    (8, 2, 128, 300, 2, 64, 4),      # the first four positions protected (TOVA+4)
    (32, 4, 128, 1100, 1, 64, 0),    # 18 state tiles, the last one ragged
])
def test_chunked_prompt_against_the_checker(H, Hkv, D, cap, B, block, keep):
    """Every token of every chunk held against the checker: dropped positions and slot tables exact, outputs
    within tolerance.  The state fills through the bulk route first, then the chunks begin."""
    w = MISTRAL.scaled(batch=B, n_q_heads=H, n_kv_heads=Hkv, head_dim=D, capacity=cap)
    n = cap + 3 * block + 30
    rep = run_lockstep(w, n, block=block, prefill_ws=True, keep_first=keep, check_state_every=1,
                       direct_fill=cap > 1000)
    assert rep.evictions == B * (n - cap)
    calls = -(-n // block)
    assert rep.cache.tova_cache_launches() < 1 + 3 * calls + 5 * (n - cap) // 8     # far fewer than 2 per token
    st = rep.cache.tova_cache_read(want_kv=True)
    q, k, v = W.tokens(w, 0, n)
    pos = st["positions"].numpy()
    for b in range(B):                    # the cached rows are the tokens the slot table names
        for s in range(0, cap, 7):
            assert np.array_equal(st["K"][b, :, s].numpy(), k[pos[b, s], b])
            assert np.array_equal(st["V"][b, :, s].numpy(), v[pos[b, s], b])


@pytest.mark.parametrize("ctas,barriers", [(-1, 0)] + [(c, nb) for c in (1, 2, 4, 8) for nb in (0, 2)])
def test_chunked_prompt_every_cluster_size(ctas, barriers):
    """The deletion kernel as one thread block reading global memory (-1) and as clusters of 1 to 8 blocks
    with staged logits, meeting once per token (the normaliser from the row sum minus the dropped rows' terms)
    or twice; capacity 333 leaves the last block of a cluster a ragged share (8 x 44 > 333)."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=333)
    rep = run_lockstep(w, 333 + 64 + 40, block=64, prefill_ws=True, chunk_cluster=ctas, check_state_every=1,
                       chunk_barriers=barriers)
    assert rep.evictions == 2 * 104
    w = LLAMA.scaled(batch=1, n_q_heads=4, n_kv_heads=4, capacity=20)      # fewer slots than blocks can share out
    rep = run_lockstep(w, 20 + 64 * 2, block=64, prefill_ws=True, chunk_cluster=ctas, check_state_every=1,
                       chunk_barriers=barriers)
    assert rep.evictions == 128
    # protected positions and a token that drops itself now and then (keep_first leaves few candidates)
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=70)
    rep = run_lockstep(w, 70 + 64 * 3 + 9, block=64, prefill_ws=True, chunk_cluster=ctas, check_state_every=1,
                       chunk_barriers=barriers, keep_first=4)
    assert rep.evictions == 2 * (64 * 3 + 9)


@pytest.mark.parametrize("keep,ctas,barriers", [(0, 0, 0), (4, 2, 0), (4, 4, 2), (0, -1, 0)])
def test_chunked_prompt_window_policy(keep, ctas, barriers):
    """Window and Window+4 on the chunked route (the row holding the earliest droppable position goes, the
    normalisers and outputs come from the same passes): every token against the checker, and the state ends up
    holding exactly the protected positions and the latest ones."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=150)
    n = 150 + 64 * 3 + 20
    rep = run_lockstep(w, n, block=64, prefill_ws=True, policy="window", keep_first=keep, chunk_cluster=ctas,
                       chunk_barriers=barriers, check_state_every=1)
    assert rep.evictions == 2 * (n - 150)
    held = rep.cache.tova_cache_read()["positions"].numpy()
    want = sorted(list(range(keep)) + list(range(n - (150 - keep), n)))
    for b in range(w.batch):
        assert sorted(held[b].tolist()) == want


def test_chunked_prompt_equals_token_by_token_processing():
    """Same prompt through the chunked route and through decode steps: the same dropped positions, the same
    state, outputs within the output tolerance; later decode steps bit-identical.  Also: no outputs wanted,
    positions from the device counter, and the route switched off again."""
    w = LLAMA.scaled(batch=2, n_q_heads=8, n_kv_heads=4, capacity=150)
    T = 150 + 64 * 3 + 20
    q, k, v = W.tokens(w, 0, T + 10)
    a, b, c = make_cache(w, prefill_ws=True), make_cache(w), make_cache(w, prefill_ws=True)
    oa, ea = gpu_block(a, w, q[:T], k[:T], v[:T], 0, use_prefill=True)
    ob, eb = gpu_block(b, w, q[:T], k[:T], v[:T], 0, use_prefill=False)
    assert np.array_equal(ea, eb)
    assert np.abs(oa - ob).max() <= out_tol(w)
    assert a.tova_cache_launches() < b.tova_cache_launches() // 4
    dq, dk, dv = (tova.to_device(x, w.dtype) for x in (q, k, v))
    ev = torch.empty(T, w.batch, dtype=torch.int32, device="cuda:0")
    c.tova_prefill(dq[:9], dk[:9], dv[:9], 9, 0, None, ev[:9])
    c.tova_prefill(dq[9:T], dk[9:T], dv[9:T], T - 9, tova.TOVA_POS_AUTO, None, ev[9:])
    torch.cuda.synchronize()
    assert np.array_equal(ev.cpu().numpy(), ea)
    a.tova_cache_set_prefill_workspace(None, allocate=False)
    o1, e1 = gpu_block(a, w, q[T:], k[T:], v[T:], T, use_prefill=True)
    o2, e2 = gpu_block(b, w, q[T:], k[T:], v[T:], T, use_prefill=False)
    o3, e3 = gpu_block(c, w, q[T:], k[T:], v[T:], T, use_prefill=False)
    assert np.array_equal(o1, o2) and np.array_equal(e1, e2) and np.array_equal(o1, o3) and np.array_equal(e1, e3)
    sa, sb, sc = (x.tova_cache_read(want_kv=True) for x in (a, b, c))
    for key in ("len", "positions", "K", "V"):
        assert torch.equal(sa[key], sb[key]) and torch.equal(sa[key], sc[key]), key
    assert sa["status"] == 0 and sc["status"] == 0


def test_prefill_workspace_argument_errors():
    w = LLAMA.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=70)
    c = make_cache(w)
    small = torch.empty(1024, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(tova.TovaError) as e:
        c.tova_cache_set_prefill_workspace(small)
    assert e.value.code == -5
    f = make_cache(W.WORKLOADS["tiny"])
    with pytest.raises(tova.TovaError):
        f.tova_cache_set_prefill_workspace()                   # fp32 states keep the per-token route
    for bad in (3, 16, -2):
        with pytest.raises(tova.TovaError):
            c.tova_cache_set_chunk_cluster(bad)
    for bad in (1, 3, -1):
        with pytest.raises(tova.TovaError):
            c.tova_cache_set_chunk_barriers(bad)
    c.tova_cache_set_chunk_barriers(2)
    c.tova_cache_set_chunk_barriers(0)


def test_bulk_prefill_mode_argument():
    c = make_cache(LLAMA.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=70))
    for mode in (0, 1, 2, True, False):
        c.tova_cache_set_bulk_prefill(mode)
    for bad in (3, -1):
        with pytest.raises(tova.TovaError):
            c.tova_cache_set_bulk_prefill(bad)


def test_bulk_prefill_against_the_checker_with_automatic_positions():
    """Bulk runs of several query tiles held against the checker token by token; positions continue from
    the device counter (TOVA_POS_AUTO) across a bulk run and the per-token steps after it."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=200)
    rep = run_lockstep(w, 200 + 60, block=150)          # runs of 150 and 50 tokens in bulk, then evictions
    assert rep.evictions == 2 * 60
    T = 230
    q, k, v = W.tokens(w, 0, T)
    c = make_cache(w)
    dq, dk, dv = (tova.to_device(x, w.dtype) for x in (q, k, v))
    ev = torch.empty(T, w.batch, dtype=torch.int32, device="cuda:0")
    c.tova_prefill(dq[:5], dk[:5], dv[:5], 5, 0, None, ev[:5])                        # position counter starts at 0
    c.tova_prefill(dq[5:], dk[5:], dv[5:], T - 5, tova.TOVA_POS_AUTO, None, ev[5:])   # no outputs wanted
    torch.cuda.synchronize()
    log = ev.cpu().numpy()
    assert np.array_equal(log, np.concatenate(rep.evicted_log)[:T])
    st = c.tova_cache_read()
    held = replay_slot_table(log, w.capacity)
    for b in range(w.batch):
        assert set(st["positions"][b].tolist()) == held[b]


def test_cached_rows_are_the_inserted_tokens():
    """tova_cache_read returns, per slot, exactly the k/v of the position it reports."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=48)
    T = 150
    q, k, v = W.tokens(w, 0, T)
    c = make_cache(w)
    gpu_block(c, w, q, k, v, 0)
    st = c.tova_cache_read(want_kv=True)
    pos = st["positions"].numpy()
    for b in range(w.batch):
        assert len(set(pos[b].tolist())) == w.capacity
        for s in range(w.capacity):
            assert np.array_equal(st["K"][b, :, s].numpy(), k[pos[b, s], b])
            assert np.array_equal(st["V"][b, :, s].numpy(), v[pos[b, s], b])


def test_sequences_are_independent_on_gpu():
    w = LLAMA.scaled(batch=3, n_q_heads=4, n_kv_heads=4, capacity=70)
    T = 200
    q, k, v = W.tokens(w, 0, T)
    full = make_cache(w)
    of, ef = gpu_block(full, w, q, k, v, 0)
    for b in range(w.batch):
        w1 = w.scaled(batch=1)
        one = make_cache(w1)
        o1, e1 = gpu_block(one, w1, q[:, b:b + 1], k[:, b:b + 1], v[:, b:b + 1], 0)
        assert np.array_equal(o1[:, 0], of[:, b]) and np.array_equal(e1[:, 0], ef[:, b])


def test_unbounded_arm_matches_checker_and_reports_full():
    w = LLAMA.scaled(batch=2, n_q_heads=4, n_kv_heads=4, capacity=150)
    cache = make_cache(w, evict=False)
    rep = run_lockstep(w, 150, cache=cache, block=50)
    assert rep.evictions == 0 and cache.tova_cache_len() == 150
    q, k, v = W.tokens(w, 150, 1)
    out = torch.empty(2, 4, 128, device="cuda:0")
    with pytest.raises(tova.TovaError) as e:
        cache.tova_decode_step(*(tova.to_device(a[0], w.dtype) for a in (q, k, v)), 150, out)
    assert e.value.code == -6


@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_entry_point_matches_device_path(pinned):
    """Page-locked buffers are read and written in place by the kernels, pageable
    ones go through staging copies: the same results either way."""
    w = LLAMA.scaled(batch=2, n_q_heads=4, n_kv_heads=4, capacity=40)
    T = 90
    q, k, v = W.tokens(w, 0, T)
    dev = make_cache(w)
    o_dev, e_dev = gpu_block(dev, w, q, k, v, 0, use_prefill=False)
    host = make_cache(w)
    pin = (lambda x: x.pin_memory()) if pinned else (lambda x: x)
    hq, hk, hv = (pin(torch.from_numpy(a).to(torch.bfloat16)) for a in (q, k, v))
    out = pin(torch.empty(w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32))
    ev = pin(torch.empty(w.batch, dtype=torch.int32))
    for t in range(T):
        host.tova_decode_step_host(hq[t], hk[t], hv[t], t, out, ev)
        assert np.array_equal(out.numpy(), o_dev[t]) and np.array_equal(ev.numpy(), e_dev[t])


def test_step_argument_errors():
    w = LLAMA.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=8)
    c = make_cache(w)
    q = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros(1, 2, 128, device="cuda:0")
    with pytest.raises(tova.TovaError) as e:
        c.tova_decode_step(q, q, None, 0, out)
    assert e.value.code == -1
    mis = torch.zeros(2 * 128 + 8, dtype=torch.bfloat16, device="cuda:0")[4:4 + 256].view(1, 2, 128)
    with pytest.raises(tova.TovaError) as e:
        c.tova_decode_step(mis, q, q, 0, out)
    assert e.value.code == -4
    with pytest.raises(tova.TovaError):
        c.tova_cache_set_chunk_rows(48)
    assert c.tova_cache_len() == 0


@pytest.mark.parametrize("fused", [True, False])
def test_deferred_eviction_gives_identical_results(fused):
    """Eviction on the cache's side stream, two caches taking turns like the
    layers of a model: same outputs, dropped positions and state as the default.
    Launches per step: streaming kernel + eviction kernel, plus the outputs-only
    kernel when the partials are merged through global memory."""
    w = LLAMA.scaled(batch=2, n_q_heads=8, n_kv_heads=4, capacity=90)
    T = 220
    streams = [W.tokens(w, 0, T, layer=l) for l in range(2)]
    ref = [make_cache(w, fused_merge=fused) for _ in range(2)]
    dfr = [make_cache(w, fused_merge=fused) for _ in range(2)]
    for c in dfr:
        c.tova_cache_set_deferred_eviction(True)
    dev = [[tova.to_device(a, w.dtype) for a in s] for s in streams]
    shape = (T, w.batch, w.n_q_heads, w.head_dim)
    o_ref = [torch.empty(shape, device="cuda:0") for _ in range(2)]
    o_dfr = [torch.empty(shape, device="cuda:0") for _ in range(2)]
    e_ref = [torch.full((T, w.batch), -7, dtype=torch.int32, device="cuda:0") for _ in range(2)]
    e_dfr = [torch.full((T, w.batch), -7, dtype=torch.int32, device="cuda:0") for _ in range(2)]
    for t in range(T):
        for l in range(2):
            q, k, v = dev[l]
            ref[l].tova_decode_step(q[t], k[t], v[t], t, o_ref[l][t], e_ref[l][t])
            dfr[l].tova_decode_step(q[t], k[t], v[t], t, o_dfr[l][t], e_dfr[l][t])
    for c in dfr:
        c.tova_cache_join()
    torch.cuda.synchronize()
    for l in range(2):
        assert torch.equal(o_ref[l], o_dfr[l]) and torch.equal(e_ref[l], e_dfr[l])
        a, b = ref[l].tova_cache_read(want_kv=True), dfr[l].tova_cache_read(want_kv=True)
        assert a["status"] == 0 and b["status"] == 0
        for key in ("len", "positions", "K", "V"):
            assert torch.equal(a[key], b[key]), key
        assert dfr[l].tova_cache_launches() == 1 + (2 if fused else 3) * T


# ---------------------------------------------------------------------------
# other compression policies on the same kernels (Section 4.1, appendix ablation)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("policy,keep", [("window", 0), ("window", 4), ("tova", 1), ("tova", 4)])
@pytest.mark.parametrize("shape", ["mha", "gqa"])
def test_policy_variants_against_the_checker(policy, keep, shape):
    """Window, Window+4, TOVA+1, TOVA+4: dropped positions and slot tables bit-exact,
    outputs within tolerance; both merge routes (capacity 150: one CTA; chunk 32)."""
    w = (LLAMA.scaled(batch=2, n_q_heads=6, n_kv_heads=6, capacity=150) if shape == "mha"
         else MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=150))
    rep = run_lockstep(w, 150 + 200, block=50, policy=policy, keep_first=keep)
    assert rep.evictions == 2 * 200
    held = rep.cache.tova_cache_read()["positions"].numpy()
    for b in range(2):
        assert set(range(keep)) <= set(held[b].tolist())
        if policy == "window":       # closed form: the first i and the most recent k - i positions
            assert sorted(held[b].tolist()) == list(range(keep)) + list(range(350 - (150 - keep), 350))
    rep = run_lockstep(w, 150 + 60, block=50, policy=policy, keep_first=keep, fused_merge=False, chunk_rows=32)
    assert rep.evictions == 2 * 60


def test_policy_hand_worked_traces_on_gpu():
    from test_oracle_pins import parse_policy_golden
    toks, _ = parse_golden()
    D = 64
    for policy, keep, steps in parse_policy_golden():
        c = tova.TovaCache(1, 2, 2, D, 3, dtype=tova.TOVA_DTYPE_FP32, sm_scale=1.0)
        c.tova_cache_set_policy({"tova": 0, "window": 1}[policy], keep)
        out = torch.empty(1, 2, D, device="cuda:0")
        ev = torch.empty(1, dtype=torch.int32, device="cuda:0")
        for (t, e, rows_after, o0, o1) in steps:
            q = np.zeros((1, 2, D), np.float32); q[..., 0] = 1.0
            k = np.zeros((1, 2, D), np.float32); v = np.zeros((1, 2, D), np.float32)
            a0, v0, a1, v1 = toks[t]
            k[0, 0, 0], k[0, 1, 0] = np.log(a0), np.log(a1)
            v[0, 0, 0], v[0, 1, 0] = v0, v1
            c.tova_decode_step(*(tova.to_device(a, 0) for a in (q, k, v)), t, out, ev)
            st = c.tova_cache_read()
            assert int(ev.item()) == e, (policy, keep, t)
            assert st["positions"][0].tolist() == rows_after, (policy, keep, t)
            o = out.cpu().numpy()
            assert abs(o[0, 0, 0] - float(o0)) <= hand_tol(float(o0)) and abs(o[0, 1, 0] - float(o1)) <= hand_tol(float(o1))


@pytest.mark.parametrize("policy,recent", [("tova_head", 0), ("h2o_layer", 0), ("h2o_head", 0), ("h2o_head", 7),
                                           ("h2o_layer", 150)])
@pytest.mark.parametrize("shape", ["mha", "gqa4", "gqa16"])
def test_unit_policies_against_the_checker(policy, recent, shape):
    """TOVA-head, H2O layer-wise and head-wise: per-unit dropped positions and slot tables bit-exact, outputs within
    tolerance, accumulated scores within 1e-5 of their size; outputs merged inside the streaming kernel (capacity 150: one thread
    block per head group) and through global memory (32-row chunks, merge off)."""
    w = {"mha": LLAMA.scaled(batch=2, n_q_heads=6, n_kv_heads=6, capacity=150),
         "gqa4": MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=150),
         "gqa16": YI.scaled(batch=1, n_q_heads=32, n_kv_heads=2, capacity=150, heavy_period=40)}[shape]
    U = 1 if policy == "h2o_layer" else w.n_kv_heads
    rep = run_lockstep_units(w, 150 + 170, policy, recent, block=80)
    assert rep.evictions == w.batch * U * 170
    held = rep.cache.tova_cache_read()["positions"].numpy().reshape(w.batch, U, -1)
    if policy.startswith("h2o"):
        window = recent or 75
        for b in range(w.batch):
            for u in range(U):
                assert set(range(320 - window, 320)) <= set(held[b, u].tolist())
                if window == 150:        # a window as large as the state: first in, first out
                    assert sorted(held[b, u].tolist()) == list(range(170, 320))
    if policy == "tova_head" and U > 1:
        assert any(set(held[b, 0].tolist()) != set(held[b, 1].tolist()) for b in range(w.batch))
    rep = run_lockstep_units(w, 150 + 50, policy, recent, block=50, fused_merge=False, chunk_rows=32)
    assert rep.evictions == w.batch * U * 50


@pytest.mark.parametrize("policy,recent", [("h2o_layer", 0), ("h2o_layer", 40), ("tova_head", 0), ("h2o_head", 0)])
def test_unit_policies_with_sliced_candidates(policy, recent):
    """A state long enough that the (unit, sequence) pairs' candidates are cut into slices of thread blocks (701
    candidates: three slices, the last one ragged, the new token in it) whose minima the last block merges: same
    dropped positions, slot tables, outputs and scores as the checker, through the filling phase and beyond."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=2, capacity=700)
    U = 1 if policy == "h2o_layer" else w.n_kv_heads
    rep = run_lockstep_units(w, 700 + 120, policy, recent, block=60)
    assert rep.evictions == w.batch * U * 120


@pytest.mark.parametrize("policy", ["tova_head", "h2o_layer", "h2o_head"])
@pytest.mark.parametrize("fused", [True, False])
def test_unit_policies_deferred_eviction_gives_identical_results(policy, fused):
    """Head-wise and H2O policies with victim choice and insert on the cache's side stream, two caches taking
    turns like the layers of a model, the caller's k and v buffers overwritten right after every call: same
    outputs, dropped positions, slot tables, rows and scores as the default mode."""
    w = MISTRAL.scaled(batch=2, n_q_heads=8, n_kv_heads=4, capacity=90)
    T = 200
    code = {"tova_head": tova.TOVA_POLICY_TOVA_HEAD, "h2o_layer": tova.TOVA_POLICY_H2O_LAYER,
            "h2o_head": tova.TOVA_POLICY_H2O_HEAD}[policy]
    U = 1 if policy == "h2o_layer" else w.n_kv_heads
    streams = [W.tokens(w, 0, T, layer=l) for l in range(2)]
    ref = [make_cache(w, fused_merge=fused) for _ in range(2)]
    dfr = [make_cache(w, fused_merge=fused) for _ in range(2)]
    for c in ref + dfr:
        c.tova_cache_set_policy(code, 0)
    for c in dfr:
        c.tova_cache_set_deferred_eviction(True)
    dev = [[tova.to_device(a, w.dtype) for a in s] for s in streams]
    shape = (T, w.batch, w.n_q_heads, w.head_dim)
    o_ref = [torch.empty(shape, device="cuda:0") for _ in range(2)]
    o_dfr = [torch.empty(shape, device="cuda:0") for _ in range(2)]
    e_ref = [torch.full((T, w.batch, U), -7, dtype=torch.int32, device="cuda:0") for _ in range(2)]
    e_dfr = [torch.full((T, w.batch, U), -7, dtype=torch.int32, device="cuda:0") for _ in range(2)]
    kbuf, vbuf = torch.empty_like(dev[0][1][0]), torch.empty_like(dev[0][2][0])
    for t in range(T):
        for l in range(2):
            q, k, v = dev[l]
            ref[l].tova_decode_step(q[t], k[t], v[t], t, o_ref[l][t], e_ref[l][t])
            kbuf.copy_(k[t]); vbuf.copy_(v[t])
            dfr[l].tova_decode_step(q[t], kbuf, vbuf, t, o_dfr[l][t], e_dfr[l][t])
            kbuf.zero_(); vbuf.zero_()          # the library keeps its own copies for the later insert
    for c in dfr:
        c.tova_cache_join()
    torch.cuda.synchronize()
    for l in range(2):
        assert torch.equal(o_ref[l], o_dfr[l]) and torch.equal(e_ref[l], e_dfr[l])
        a, b = ref[l].tova_cache_read(want_kv=True), dfr[l].tova_cache_read(want_kv=True)
        assert a["status"] == 0 and b["status"] == 0
        for key in ("len", "positions", "K", "V"):
            assert torch.equal(a[key], b[key]), key
        if policy.startswith("h2o"):
            assert torch.equal(ref[l].tova_cache_read_scores(), dfr[l].tova_cache_read_scores())


def test_unit_policy_hand_worked_traces_on_gpu():
    from test_oracle_unit_policies import parse_unit_golden
    toks, _ = parse_golden()
    D = 64
    for policy, recent, steps in parse_unit_golden():
        c = tova.TovaCache(1, 2, 2, D, 3, dtype=tova.TOVA_DTYPE_FP32, sm_scale=1.0)
        c.tova_cache_set_policy({"tova_head": 2, "h2o_layer": 3, "h2o_head": 4}[policy], recent)
        U = c.tova_cache_units()
        out = torch.empty(1, 2, D, device="cuda:0")
        ev = torch.empty(1, U, dtype=torch.int32, device="cuda:0")
        for (t, e, rows_after, o0, o1) in steps:
            q = np.zeros((1, 2, D), np.float32); q[..., 0] = 1.0
            k = np.zeros((1, 2, D), np.float32); v = np.zeros((1, 2, D), np.float32)
            a0, v0, a1, v1 = toks[t]
            k[0, 0, 0], k[0, 1, 0] = np.log(a0), np.log(a1)
            v[0, 0, 0], v[0, 1, 0] = v0, v1
            c.tova_decode_step(*(tova.to_device(a, 0) for a in (q, k, v)), t, out, ev)
            st = c.tova_cache_read()
            assert ev.cpu().numpy()[0].tolist() == e, (policy, recent, t)
            assert st["positions"].numpy().reshape(U, 3).tolist() == rows_after, (policy, recent, t)
            o = out.cpu().numpy()
            assert abs(o[0, 0, 0] - float(o0)) <= hand_tol(float(o0)) and abs(o[0, 1, 0] - float(o1)) <= hand_tol(float(o1))
            assert st["status"] == 0


# ---------------------------------------------------------------------------
# position compression (Section "Extrapolation with TOVA")
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("H,Hkv,D,dtype,cap,B,policy,keep", [
    (8, 8, 128, W.DTYPE_BF16, 64, 2, "tova", 0),      # MHA
    (8, 2, 128, W.DTYPE_BF16, 100, 2, "tova", 2),     # GQA 4, two protected positions
    (16, 1, 64, W.DTYPE_BF16, 70, 1, "tova", 0),      # GQA 16 (four head groups per KV head), D = 64
    (4, 4, 64, W.DTYPE_FP32, 48, 2, "tova", 0),       # fp32
    (4, 2, 128, W.DTYPE_FP32, 40, 1, "window", 4),    # Window+4 on compressed positions
])
def test_position_compression_against_the_checker(H, Hkv, D, dtype, cap, B, policy, keep):
    """q and k come without rotary embedding; 500 tokens through a small state leave retained tokens hundreds of
    positions apart, so the ln ln rule is at work in almost every step.  Dropped positions and slot tables exact,
    outputs within tolerance, and the compressed positions of the last step equal to the checker's."""
    w = MISTRAL.scaled(batch=B, n_q_heads=H, n_kv_heads=Hkv, head_dim=D, dtype=dtype, capacity=cap)
    assert not w.rope
    rep = run_lockstep(w, 500, block=50, rope_base=10000.0, policy=policy, keep_first=keep)
    assert rep.evictions == B * (500 - cap)
    cp = rep.cache.tova_cache_read_compressed_positions().numpy()
    assert np.abs(cp - rep.oracle.last_cpos).max() < 1e-9
    pos = rep.cache.tova_cache_read()["positions"].numpy()
    assert max(np.diff(np.sort(pos[0]))) > 10                      # gaps above 10 were there to compress
    assert rep.cache.tova_cache_launches() == 1 + 3 * 500


def test_position_compression_argument_errors():
    w = MISTRAL.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=8)
    c = make_cache(w)
    with pytest.raises(tova.TovaError) as e:
        c.tova_cache_read_compressed_positions()
    assert e.value.code == -3
    q = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda:0")
    c.tova_decode_step(q, q, q, 0, torch.zeros(1, 2, 128, device="cuda:0"))
    with pytest.raises(tova.TovaError):            # keys already cached: too late to switch
        c.tova_cache_set_position_compression(10000.0)
    big = make_cache(MISTRAL.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=20000))
    with pytest.raises(tova.TovaError) as e:
        big.tova_cache_set_position_compression(10000.0)
    assert e.value.code == -3
    d = make_cache(w)
    d.tova_cache_set_position_compression(10000.0)
    with pytest.raises(tova.TovaError):
        d.tova_cache_set_policy(tova.TOVA_POLICY_TOVA_HEAD, 0)
    d.tova_cache_set_position_compression(on=False)
    d.tova_cache_set_policy(tova.TOVA_POLICY_TOVA_HEAD, 0)


def test_policy_argument_errors():
    w = LLAMA.scaled(batch=1, n_q_heads=2, n_kv_heads=2, capacity=8)
    c = make_cache(w)
    with pytest.raises(tova.TovaError) as e:
        c.tova_cache_set_policy(7, 0)
    assert e.value.code == -3
    for bad in (-1, 8):
        with pytest.raises(tova.TovaError):
            c.tova_cache_set_policy(tova.TOVA_POLICY_WINDOW, bad)
    with pytest.raises(tova.TovaError):
        c.tova_cache_set_policy(tova.TOVA_POLICY_TOVA_HEAD, 1)       # the per-head policy takes no argument
    with pytest.raises(tova.TovaError):
        c.tova_cache_set_policy(tova.TOVA_POLICY_H2O_HEAD, 9)        # a window larger than the state
    with pytest.raises(tova.TovaError) as e:
        c.tova_cache_read_scores()                                   # scores exist under H2O only
    assert e.value.code == -3
    c.tova_cache_set_policy(tova.TOVA_POLICY_H2O_LAYER, 0)
    assert c.tova_cache_units() == 1
    c.tova_cache_set_policy(tova.TOVA_POLICY_TOVA_HEAD, 0)
    assert c.tova_cache_units() == 2
    c.tova_cache_set_policy(tova.TOVA_POLICY_WINDOW, 7)
    assert c.tova_cache_units() == 1
    q = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda:0")
    c.tova_decode_step(q, q, q, 0, torch.zeros(1, 2, 128, device="cuda:0"))
    with pytest.raises(tova.TovaError):            # the state is no longer empty
        c.tova_cache_set_policy(tova.TOVA_POLICY_TOVA, 0)
