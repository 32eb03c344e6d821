"""Thin ctypes binding of the C ABI in include/tova.h.

Argument marshalling only: every step of the decode path runs in the CUDA
library.  torch is used for device memory and streams.  Loading fails loudly
if the library has not been built; nothing here computes on the CPU.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

TOVA_DTYPE_FP32 = 0
TOVA_DTYPE_BF16 = 1
TOVA_POLICY_TOVA = 0
TOVA_POLICY_WINDOW = 1
TOVA_POLICY_TOVA_HEAD = 2
TOVA_POLICY_H2O_LAYER = 3
TOVA_POLICY_H2O_HEAD = 4
TOVA_POS_AUTO = -1       # "the previous token's position + 1"


class TovaError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: status {code} ({strerror(code)})")
        self.code = code


class tova_config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("capacity", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("sm_scale", ctypes.c_float), ("evict", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded CUDA library (built on first use if nvcc is present)."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            path = _build.build()
        L = ctypes.CDLL(path)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.tova_cache_bytes.restype = ctypes.c_size_t
        L.tova_cache_bytes.argtypes = [ctypes.POINTER(tova_config)]
        L.tova_cache_init.restype = ctypes.c_int
        L.tova_cache_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(tova_config), vp,
                                      ctypes.c_size_t, vp]
        L.tova_decode_step.restype = ctypes.c_int
        L.tova_decode_step.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp]
        L.tova_prefill.restype = ctypes.c_int
        L.tova_prefill.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp]
        L.tova_decode_step_host.restype = ctypes.c_int
        L.tova_decode_step_host.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp]
        L.tova_cache_read.restype = ctypes.c_int
        L.tova_cache_read.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.tova_cache_set_chunk_rows.restype = ctypes.c_int
        L.tova_cache_set_chunk_rows.argtypes = [vp, i32]
        L.tova_cache_set_policy.restype = ctypes.c_int
        L.tova_cache_set_policy.argtypes = [vp, i32, i32]
        L.tova_prefill_workspace_bytes.restype = ctypes.c_size_t
        L.tova_prefill_workspace_bytes.argtypes = [ctypes.POINTER(tova_config)]
        L.tova_cache_set_prefill_workspace.restype = ctypes.c_int
        L.tova_cache_set_prefill_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        L.tova_position_workspace_bytes.restype = ctypes.c_size_t
        L.tova_position_workspace_bytes.argtypes = [ctypes.POINTER(tova_config)]
        L.tova_cache_set_position_compression.restype = ctypes.c_int
        L.tova_cache_set_position_compression.argtypes = [vp, vp, ctypes.c_size_t, ctypes.c_float]
        L.tova_cache_read_compressed_positions.restype = ctypes.c_int
        L.tova_cache_read_compressed_positions.argtypes = [vp, vp, vp]
        L.tova_shard_table_bytes.restype = ctypes.c_size_t
        L.tova_shard_table_bytes.argtypes = [ctypes.POINTER(tova_config), i32]
        L.tova_cache_set_shard.restype = ctypes.c_int
        L.tova_cache_set_shard.argtypes = [vp, i32, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp)]
        L.tova_decode_step_scores.restype = ctypes.c_int
        L.tova_decode_step_scores.argtypes = [vp, vp, vp, vp, i32, vp, vp]
        L.tova_decode_step_commit.restype = ctypes.c_int
        L.tova_decode_step_commit.argtypes = [vp, vp, vp, vp, vp]
        L.tova_cache_set_chunk_cluster.restype = ctypes.c_int
        L.tova_cache_set_chunk_cluster.argtypes = [vp, i32]
        L.tova_cache_set_chunk_barriers.restype = ctypes.c_int
        L.tova_cache_set_chunk_barriers.argtypes = [vp, i32]
        L.tova_cache_read_scores.restype = ctypes.c_int
        L.tova_cache_read_scores.argtypes = [vp, vp, vp]
        L.tova_cache_units.restype = i32
        L.tova_cache_units.argtypes = [vp]
        L.tova_cache_set_fused_merge.restype = ctypes.c_int
        L.tova_cache_set_fused_merge.argtypes = [vp, i32]
        L.tova_cache_set_bulk_prefill.restype = ctypes.c_int
        L.tova_cache_set_bulk_prefill.argtypes = [vp, i32]
        L.tova_cache_set_deferred_eviction.restype = ctypes.c_int
        L.tova_cache_set_deferred_eviction.argtypes = [vp, i32]
        L.tova_cache_join.restype = ctypes.c_int
        L.tova_cache_join.argtypes = [vp, vp]
        L.tova_cache_len.restype = i32
        L.tova_cache_len.argtypes = [vp]
        L.tova_cache_launches.restype = i64
        L.tova_cache_launches.argtypes = [vp]
        L.tova_cache_destroy.restype = ctypes.c_int
        L.tova_cache_destroy.argtypes = [vp]
        L.tova_decode_step_static.restype = ctypes.c_int
        L.tova_decode_step_static.argtypes = [ctypes.POINTER(tova_config), vp, vp, vp, i32, vp, vp, vp,
                                              i32, vp, vp, vp, vp]
        L.tova_strerror.restype = ctypes.c_char_p
        L.tova_strerror.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().tova_strerror(int(code)).decode()


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise TovaError(rc, what)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def tova_cache_bytes(cfg: tova_config) -> int:
    return int(lib().tova_cache_bytes(ctypes.byref(cfg)))


class TovaCache:
    """State of one layer for `batch` sequences; the names follow the C ABI."""

    def __init__(self, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, capacity: int,
                 dtype: int = TOVA_DTYPE_BF16, sm_scale: float = 0.0, evict: bool = True,
                 device: str = "cuda:0", stream: Optional[torch.cuda.Stream] = None):
        self.cfg = tova_config(batch, n_q_heads, n_kv_heads, head_dim, capacity, dtype,
                               float(sm_scale), 1 if evict else 0)
        nbytes = tova_cache_bytes(self.cfg)
        if nbytes == 0:
            raise TovaError(-2, "tova_cache_bytes rejected the configuration")
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if dtype == TOVA_DTYPE_BF16 else torch.float32
        self.nbytes = nbytes
        with torch.cuda.device(self.device):
            self.mem = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            off = (-self.mem.data_ptr()) % 256
            self._base = self.mem.data_ptr() + off
            h = ctypes.c_void_p()
            _check(lib().tova_cache_init(ctypes.byref(h), ctypes.byref(self.cfg),
                                         ctypes.c_void_p(self._base), nbytes, _stream(stream)),
                   "tova_cache_init")
        self._h = h

    # -- C ABI calls ---------------------------------------------------------
    def tova_decode_step(self, q, k, v, pos: int, out, evicted_pos=None, stream=None) -> None:
        _check(lib().tova_decode_step(self._h, _p(q), _p(k), _p(v), int(pos), _p(out),
                                      _p(evicted_pos), _stream(stream)), "tova_decode_step")

    def tova_prefill(self, q, k, v, n_tokens: int, first_pos: int, out=None, evicted_pos=None,
                     stream=None) -> None:
        _check(lib().tova_prefill(self._h, _p(q), _p(k), _p(v), int(n_tokens), int(first_pos),
                                  _p(out), _p(evicted_pos), _stream(stream)), "tova_prefill")

    def tova_decode_step_host(self, q, k, v, pos: int, out, evicted_pos=None, stream=None) -> None:
        """q, k, v, out, evicted_pos are HOST tensors (pinned for async copies)."""
        _check(lib().tova_decode_step_host(self._h, _p(q), _p(k), _p(v), int(pos), _p(out),
                                           _p(evicted_pos), _stream(stream)), "tova_decode_step_host")

    def tova_cache_read(self, want_kv: bool = False, stream=None):
        """Returns dict(len [B], positions [B,cap], status int, K, V or None) on the host."""
        c = self.cfg
        ln = torch.empty(c.batch, dtype=torch.int32, device=self.device)
        units = self.tova_cache_units()
        ps = (torch.empty(c.batch, c.capacity, dtype=torch.int32, device=self.device) if units == 1 else
              torch.empty(c.batch, units, c.capacity, dtype=torch.int32, device=self.device))
        stt = torch.empty(1, dtype=torch.int32, device=self.device)
        K = V = None
        if want_kv:
            K = torch.empty(c.batch, c.n_kv_heads, c.capacity, c.head_dim, dtype=self.tdtype,
                            device=self.device)
            V = torch.empty_like(K)
        _check(lib().tova_cache_read(self._h, _p(ln), _p(ps), _p(K), _p(V), _p(stt), _stream(stream)),
               "tova_cache_read")
        torch.cuda.synchronize(self.device)
        return {"len": ln.cpu(), "positions": ps.cpu(), "status": int(stt.item()),
                "K": None if K is None else K.float().cpu(), "V": None if V is None else V.float().cpu()}

    def tova_cache_set_prefill_workspace(self, mem: Optional[torch.Tensor] = None, allocate: bool = True):
        """Gives the cache the scratch of the chunked prompt route: `mem`, a uint8 device tensor the caller
        keeps alive (it may serve several caches of one shape), or a fresh one when allocate is set.
        mem=None with allocate=False switches the route off.  Returns the tensor in use."""
        if mem is None and not allocate:
            _check(lib().tova_cache_set_prefill_workspace(self._h, None, 0), "tova_cache_set_prefill_workspace")
            self._prefill_ws = None
            return None
        need = int(lib().tova_prefill_workspace_bytes(ctypes.byref(self.cfg)))
        if need == 0:
            raise TovaError(-3, "tova_prefill_workspace_bytes rejected the configuration")
        if mem is None:
            mem = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        off = (-mem.data_ptr()) % 256
        _check(lib().tova_cache_set_prefill_workspace(self._h, ctypes.c_void_p(mem.data_ptr() + off),
                                                      mem.numel() - off), "tova_cache_set_prefill_workspace")
        self._prefill_ws = mem
        return mem

    def tova_cache_set_position_compression(self, rope_base: float = 10000.0, on: bool = True) -> None:
        """Switches the position compression on (allocating its workspace) or off; callers then pass q and k
        without rotary embedding."""
        if not on:
            _check(lib().tova_cache_set_position_compression(self._h, None, 0, 0.0), "tova_cache_set_position_compression")
            self._poscomp_ws = None
            return
        need = int(lib().tova_position_workspace_bytes(ctypes.byref(self.cfg)))
        mem = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        off = (-mem.data_ptr()) % 256
        _check(lib().tova_cache_set_position_compression(self._h, ctypes.c_void_p(mem.data_ptr() + off), need,
                                                         float(rope_base)), "tova_cache_set_position_compression")
        self._poscomp_ws = mem

    def tova_cache_read_compressed_positions(self, stream=None):
        c = self.cfg
        cp = torch.empty(c.batch, c.capacity + 1, dtype=torch.float64, device=self.device)
        _check(lib().tova_cache_read_compressed_positions(self._h, _p(cp), _stream(stream)),
               "tova_cache_read_compressed_positions")
        torch.cuda.synchronize(self.device)
        return cp.cpu()

    def tova_shard_table_bytes(self, world: int) -> int:
        return int(lib().tova_shard_table_bytes(ctypes.byref(self.cfg), int(world)))

    def tova_cache_set_shard(self, rank: int, world: int, n_q_heads_total: int, peer_tables, peer_flags=None) -> None:
        """peer_tables / peer_flags: lists of `world` device tensors (or data pointers) as mapped into this process;
        peer_flags None = the caller sums peer_tables[rank] over the ranks between scores and commit."""
        def ptrs(xs):
            arr = (ctypes.c_void_p * world)()
            for i, x in enumerate(xs):
                arr[i] = None if x is None else (x.data_ptr() if hasattr(x, "data_ptr") else int(x))
            return arr
        tabs = ptrs(peer_tables)
        flags = None if peer_flags is None else ptrs(peer_flags)
        self._shard_keep = (peer_tables, peer_flags)
        _check(lib().tova_cache_set_shard(self._h, int(rank), int(world), int(n_q_heads_total), tabs, flags),
               "tova_cache_set_shard")

    def tova_decode_step_scores(self, q, k, v, pos: int, out, stream=None) -> None:
        _check(lib().tova_decode_step_scores(self._h, _p(q), _p(k), _p(v), int(pos), _p(out), _stream(stream)),
               "tova_decode_step_scores")

    def tova_decode_step_commit(self, k, v, evicted_pos=None, stream=None) -> None:
        _check(lib().tova_decode_step_commit(self._h, _p(k), _p(v), _p(evicted_pos), _stream(stream)),
               "tova_decode_step_commit")

    def tova_cache_set_chunk_cluster(self, ctas: int) -> None:
        _check(lib().tova_cache_set_chunk_cluster(self._h, int(ctas)), "tova_cache_set_chunk_cluster")

    def tova_cache_set_chunk_barriers(self, per_token: int) -> None:
        _check(lib().tova_cache_set_chunk_barriers(self._h, int(per_token)), "tova_cache_set_chunk_barriers")

    def tova_cache_set_chunk_rows(self, rows: int) -> None:
        _check(lib().tova_cache_set_chunk_rows(self._h, int(rows)), "tova_cache_set_chunk_rows")

    def tova_cache_set_policy(self, policy: int, arg: int = 0) -> None:
        """policy: one of TOVA_POLICY_*; arg = i of the "+i" variants, or the recent window of H2O."""
        _check(lib().tova_cache_set_policy(self._h, int(policy), int(arg)), "tova_cache_set_policy")

    def tova_cache_units(self) -> int:
        return int(lib().tova_cache_units(self._h))

    def tova_cache_read_scores(self, stream=None):
        """H2O: accumulated attention weight of every slot, [B,U,cap] on the host."""
        c = self.cfg
        sc = torch.empty(c.batch, self.tova_cache_units() if self.tova_cache_units() > 1 else 1, c.capacity,
                         dtype=torch.float32, device=self.device)
        _check(lib().tova_cache_read_scores(self._h, _p(sc), _stream(stream)), "tova_cache_read_scores")
        torch.cuda.synchronize(self.device)
        return sc.cpu()

    def tova_cache_set_fused_merge(self, on: bool) -> None:
        _check(lib().tova_cache_set_fused_merge(self._h, 1 if on else 0), "tova_cache_set_fused_merge")

    def tova_cache_set_bulk_prefill(self, mode) -> None:
        """0 / False: prompt tokens one at a time; 1 / True: bulk fill (tcgen05 kernel where head_dim is 128);
        2: bulk fill with the warp-level MMA kernel."""
        _check(lib().tova_cache_set_bulk_prefill(self._h, int(mode)), "tova_cache_set_bulk_prefill")

    def tova_cache_set_deferred_eviction(self, on: bool) -> None:
        _check(lib().tova_cache_set_deferred_eviction(self._h, 1 if on else 0),
               "tova_cache_set_deferred_eviction")

    def tova_cache_join(self, stream=None) -> None:
        _check(lib().tova_cache_join(self._h, _stream(stream)), "tova_cache_join")

    def tova_cache_len(self) -> int:
        return int(lib().tova_cache_len(self._h))

    def tova_cache_launches(self) -> int:
        return int(lib().tova_cache_launches(self._h))

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            lib().tova_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def tova_decode_step_static(cfg: tova_config, K, V, positions, n_live: int, q, k, v, pos: int, out,
                            evicted_pos=None, status=None, stream=None) -> None:
    """One decode step on caller-held state tensors, using the scratch array
    built into the library instead of a workspace: for callers that may not
    allocate device memory (see include/tova.h).  K, V [B,Hkv,cap,D] and
    positions [B,cap] are updated in place; the caller tracks n_live.  status: an
    int32 device tensor of one element that receives 0 or a device-side check's code."""
    _check(lib().tova_decode_step_static(ctypes.byref(cfg), _p(K), _p(V), _p(positions), int(n_live),
                                         _p(q), _p(k), _p(v), int(pos), _p(out), _p(evicted_pos),
                                         _p(status), _stream(stream)), "tova_decode_step_static")


def to_device(x, dtype: int, device="cuda:0") -> torch.Tensor:
    """Upload a float32 numpy array (bf16-representable for bf16) in the cache dtype."""
    t = torch.from_numpy(x)
    if dtype == TOVA_DTYPE_BF16:
        t = t.to(torch.bfloat16)
    return t.to(device)
