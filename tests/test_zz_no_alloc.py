"""tova_decode_step_static: the decode step for callers that cannot allocate.

Some users of this library run where device memory cannot be requested: inside
another engine's plugin or callback (the engine owns the allocator), in the
middle of a stream capture, or under a memory budget fixed at start-up.  They
hold the K/V tensors but cannot provide the workspace tova_cache_init wants.
tova_decode_step_static keeps the kernels' scratch in an 8 MiB array compiled
into the library instead.

The test feeds the same tokens to a regular cache (tova_decode_step) and to
the static entry point, call after call on the same shared array, across the
point where the state fills up and eviction starts, and compares outputs,
dropped positions and the final state.  The file sorts last so that a run that
stops at the first failure has already run every other test; it passes alone in
a fresh process as well as after the others, because the entry point clears the
part of the array that has to start at zero.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2401_06104_b200 as tova
from paper_2401_06104_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_both(w, n_tokens):
    dev = "cuda:0"
    tdt = torch.bfloat16 if w.dtype == W.DTYPE_BF16 else torch.float32
    q, k, v = W.tokens(w, 0, n_tokens)
    dq, dk, dv = (tova.to_device(a, w.dtype, dev) for a in (q, k, v))
    ref = tova.TovaCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, dtype=w.dtype)
    cfg = tova.tova_config(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.dtype, 0.0, 1)
    # the static caller's own state tensors (allocated here by the test, not by the call)
    K = torch.zeros(w.batch, w.n_kv_heads, w.capacity, w.head_dim, dtype=tdt, device=dev)
    V = torch.zeros_like(K)
    P = torch.full((w.batch, w.capacity), -1, dtype=torch.int32, device=dev)
    o_ref = torch.empty(w.batch, w.n_q_heads, w.head_dim, device=dev)
    o_st = torch.empty_like(o_ref)
    e_ref = torch.empty(w.batch, dtype=torch.int32, device=dev)
    e_st = torch.empty_like(e_ref)
    status = torch.full((1,), 77, dtype=torch.int32, device=dev)
    tol = 2e-3 if w.dtype == W.DTYPE_BF16 else 1e-5
    n_live = 0
    for t in range(n_tokens):
        ref.tova_decode_step(dq[t], dk[t], dv[t], t, o_ref, e_ref)
        tova.tova_decode_step_static(cfg, K, V, P, n_live, dq[t], dk[t], dv[t], t, o_st, e_st,
                                     status if t % 2 == 0 else None)
        n_live = min(n_live + 1, w.capacity)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, t
        assert float((o_ref - o_st).abs().max()) <= tol, t
        assert torch.equal(e_ref, e_st), t
    st = ref.tova_cache_read(want_kv=True)
    assert st["status"] == 0
    assert torch.equal(st["positions"], P.cpu())
    assert torch.equal(st["K"], K.float().cpu()) and torch.equal(st["V"], V.float().cpu())


def test_static_step_matches_cache_step_call_after_call():
    w = W.WORKLOADS["llama2_7b_layer"].scaled(batch=2, n_q_heads=8, n_kv_heads=4, capacity=70)
    run_both(w, 70 + 60)


def test_static_step_again_with_another_shape_on_the_same_array():
    """A second shape right after the first: whatever the previous calls left in
    the shared array must not matter."""
    w = W.WORKLOADS["tiny_unit"].scaled(batch=3, capacity=33)
    run_both(w, 33 + 40)


def test_static_step_on_the_tensor_core_kernel_with_caller_held_state():
    """Query groups of 4 and more (bf16) take the tensor-core streaming kernel, which reads the state through
    tiled tensor maps: the call encodes them over the caller's K and V every time.  Capacity 70 is not a multiple
    of the 16-row tile, and the run crosses from filling to evicting."""
    w = W.WORKLOADS["mistral_7b_gqa"].scaled(batch=3, n_q_heads=8, n_kv_heads=2, capacity=70)
    run_both(w, 70 + 50)
    w = W.WORKLOADS["yi_6b_long"].scaled(batch=1, n_q_heads=16, n_kv_heads=1, capacity=300)   # 16 heads: two N tiles
    run_both(w, 300 + 30)


def test_static_step_refuses_shapes_beyond_its_array():
    cfg = tova.tova_config(64, 32, 32, 128, 4096, tova.TOVA_DTYPE_BF16, 0.0, 1)
    one = ctypes.c_void_p(256)
    rc = tova.lib().tova_decode_step_static(ctypes.byref(cfg), one, one, one, 0, one, one, one, 0, one, None, None, None)
    assert rc == -9
    assert "8 MiB" in tova.strerror(rc)
