"""The exchange of the KV-head-sharded layer, among CPU ranks (gloo, world size 2): every rank holds half of the
heads in a checker state of its own, the ranks all-reduce their partial head sums (one vector of capacity+1
entries), take the arg-min and drop that row - and end up, token after token, with the rows, dropped positions
and outputs of the whole layer under Algorithm 1."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q_out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle.tova_oracle import OracleCache
    from test_oracle_pins import random_stream
    dist.init_process_group("gloo", rank=rank, world_size=world)
    H, Hkv, D, cap, T = 8, 4, 16, 12, 90
    Hl, Kl = H // world, Hkv // world
    q, k, v = random_stream(7, T, H, Hkv, D)                      # the same stream on every rank
    whole = OracleCache(1, H, Hkv, D, cap, precision="f64")        # the unsharded layer, for comparison
    mine = OracleCache(1, Hl, Kl, D, cap, precision="f64")
    log = []
    for t in range(T):
        ql, kl, vl = q[t, rank * Hl:(rank + 1) * Hl], k[t, rank * Kl:(rank + 1) * Kl], v[t, rank * Kl:(rank + 1) * Kl]
        forced = None
        if mine.len[0] == cap:
            # this rank's partial head sum, from a throw-away copy of its state (the step itself comes after the exchange)
            probe = OracleCache(1, Hl, Kl, D, cap, precision="f64")
            probe.len[:], probe.pos[:], probe.K[:], probe.V[:] = mine.len, mine.pos, mine.K, mine.V
            *_, mean_local = probe.step(ql[None], kl[None], vl[None], t, want_mean=True)
            part = torch.from_numpy(mean_local[0] * (Hl / H))      # sum over local heads / H_total
            dist.all_reduce(part, op=dist.ReduceOp.SUM)            # the one exchange: capacity+1 numbers
            forced = np.array([int(np.argmin(part.numpy()))], np.int32)   # numpy: first minimum = lowest slot
        out, ev, *_ = mine.step(ql[None], kl[None], vl[None], t, forced=forced)
        o_w, e_w, *_ = whole.step(q[t][None], k[t][None], v[t][None], t)
        assert ev[0] == e_w[0], (t, ev, e_w)
        assert np.abs(out[0] - o_w[0, rank * Hl:(rank + 1) * Hl]).max() < 1e-12
        assert np.array_equal(mine.pos, whole.pos)
        assert np.array_equal(mine.K[0], whole.K[0, rank * Kl:(rank + 1) * Kl])
        log.append(int(ev[0]))
    gathered = [None] * world
    dist.all_gather_object(gathered, log)
    assert all(g == log for g in gathered)                         # every rank dropped the same positions
    q_out.put((rank, sum(1 for e in log if e >= 0)))
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_layer_policy_through_one_small_all_reduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 78, 1: 78}                                   # 90 tokens, capacity 12: 78 drops on both ranks
