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
    check_all_sequences(rep, w, n)
    print(f"{name} k={cap}: max_err {rep.max_err:.2e} resyncs {rep.resyncs}/{rep.evictions} "
          f"self {rep.self_evictions}")
