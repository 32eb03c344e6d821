"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function the header declares, sizes its device block sensibly and
rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest
import torch

import paper_2401_06104_b200 as tova
from paper_2401_06104_b200 import build as tbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def cfg(**kw):
    base = dict(batch=2, n_q_heads=8, n_kv_heads=4, head_dim=128, capacity=100,
                dtype=tova.TOVA_DTYPE_BF16, sm_scale=0.0, evict=1)
    base.update(kw)
    return tova.tova_config(**base)


def test_library_builds_and_exports_every_declared_symbol():
    tbuild.build()
    L = tova.lib()
    header = open(os.path.join(ROOT, "include", "tova.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(tova_[a-z_0-9]+)\s*\(", header))
    assert {"tova_cache_init", "tova_prefill", "tova_decode_step", "tova_cache_read"} <= names
    for n in names:
        assert hasattr(L, n), n


def test_cache_bytes_counts_state_and_scratch():
    c = cfg()
    n = tova.tova_cache_bytes(c)
    kv = 2 * 2 * 4 * 100 * 128 * 2
    assert n > kv
    assert n < kv + 4 * 1024 * 1024
    big = tova.tova_cache_bytes(cfg(batch=8, n_q_heads=32, n_kv_heads=32, capacity=512))
    assert 64 * 2**20 < big < 80 * 2**20          # 64 MiB of K/V plus scratch


def test_prefill_workspace_size_is_dominated_by_the_logits():
    c = cfg(batch=4, n_q_heads=8, n_kv_heads=2, capacity=1000)
    n = tova.lib().tova_prefill_workspace_bytes(ctypes.byref(c))
    logits = 4 * 8 * 64 * (1000 + 64) * 4
    assert logits < n < logits + 2 * 2**20
    assert tova.lib().tova_prefill_workspace_bytes(ctypes.byref(cfg(dtype=tova.TOVA_DTYPE_FP32))) == 0
    assert tova.lib().tova_prefill_workspace_bytes(ctypes.byref(cfg(capacity=0))) == 0


@pytest.mark.parametrize("bad", [dict(batch=0), dict(n_q_heads=6), dict(capacity=0), dict(n_kv_heads=0),
                                 dict(head_dim=96), dict(dtype=7), dict(sm_scale=-1.0)])
def test_invalid_configurations_are_rejected(bad):
    assert tova.tova_cache_bytes(cfg(**bad)) == 0
    h = ctypes.c_void_p()
    rc = tova.lib().tova_cache_init(ctypes.byref(h), ctypes.byref(cfg(**bad)), ctypes.c_void_p(256), 1 << 30, None)
    assert rc in (-2, -3) and not h.value


def test_init_argument_errors_come_before_any_cuda_call():
    L = tova.lib()
    c = cfg()
    need = tova.tova_cache_bytes(c)
    h = ctypes.c_void_p()
    assert L.tova_cache_init(None, ctypes.byref(c), ctypes.c_void_p(256), need, None) == -1
    assert L.tova_cache_init(ctypes.byref(h), None, ctypes.c_void_p(256), need, None) == -1
    assert L.tova_cache_init(ctypes.byref(h), ctypes.byref(c), None, need, None) == -1
    assert L.tova_cache_init(ctypes.byref(h), ctypes.byref(c), ctypes.c_void_p(264), need, None) == -4
    assert L.tova_cache_init(ctypes.byref(h), ctypes.byref(c), ctypes.c_void_p(256), need - 1, None) == -5
    assert not h.value


def test_null_handles_are_rejected():
    L = tova.lib()
    assert L.tova_decode_step(None, None, None, None, 0, None, None, None) == -1
    assert L.tova_prefill(None, None, None, None, 1, 0, None, None, None) == -1
    assert L.tova_decode_step_host(None, None, None, None, 0, None, None, None) == -1
    assert L.tova_cache_read(None, None, None, None, None, None, None) == -1
    assert L.tova_cache_destroy(None) == -1
    assert L.tova_cache_len(None) == -1
    assert L.tova_cache_set_bulk_prefill(None, 1) == -1
    assert L.tova_cache_set_policy(None, 2, 0) == -1
    assert L.tova_cache_read_scores(None, None, None) == -1
    assert L.tova_cache_units(None) == -1
    assert L.tova_cache_set_prefill_workspace(None, None, 0) == -1
    assert L.tova_cache_set_chunk_cluster(None, 0) == -1
    assert L.tova_cache_set_chunk_barriers(None, 0) == -1
    assert L.tova_cache_set_position_compression(None, None, 0, 10000.0) == -1
    assert L.tova_cache_read_compressed_positions(None, None, None) == -1
    assert L.tova_position_workspace_bytes(ctypes.byref(cfg())) > 2 * 101 * 64 * 8
    assert L.tova_cache_set_shard(None, 0, 1, 8, None, None) == -1
    assert L.tova_decode_step_scores(None, None, None, None, 0, None, None) == -1
    assert L.tova_decode_step_commit(None, None, None, None, None) == -1
    c = cfg()
    assert L.tova_shard_table_bytes(ctypes.byref(c), 2) == 2 * 2 * 2 * 104 * 4 and L.tova_shard_table_bytes(ctypes.byref(c), 9) == 0
    assert tova.strerror(0) == "ok" and "aligned" in tova.strerror(-4)


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a GPU")
def test_no_cpu_fallback_without_a_device():
    """Valid arguments but no CUDA device: the call fails, nothing is emulated."""
    c = cfg()
    h = ctypes.c_void_p()
    rc = tova.lib().tova_cache_init(ctypes.byref(h), ctypes.byref(c), ctypes.c_void_p(256),
                                    tova.tova_cache_bytes(c), None)
    assert rc == -7 and not h.value
