"""Pins for the checker's position compression (Section "Extrapolation with TOVA": the gap g between
neighbouring retained tokens becomes ln(ln(g)), unchanged while g <= 10; keys are cached without rotary
embedding, which is applied with the compressed positions at every step).

Compared with things other than the checker: the values the paper's rule gives on worked gaps, a library
attention routine on the case where nothing is compressed, an invariance rotary embedding has, and a
restatement over the full token history written with complex exponentials in float64."""
import math

import numpy as np
import pytest
import torch

from oracle.tova_oracle import OracleCache, compress_gap
from test_oracle_pins import random_stream, softmax64

BASE = 10000.0


def rope_complex(x, p, base=BASE):
    """Rotary embedding of x [..., D] at (real) position p: pairs (d, d + D/2) as complex numbers times
    exp(i p base^(-2d/D)).  float64."""
    D = x.shape[-1]
    half = D // 2
    z = x[..., :half].astype(np.float64) + 1j * x[..., half:].astype(np.float64)
    z = z * np.exp(1j * p * BASE ** (-2.0 * np.arange(half) / D) if base == BASE else
                   1j * p * base ** (-2.0 * np.arange(half) / D))
    return np.concatenate([z.real, z.imag], axis=-1)


def chain(positions):
    """Compressed positions of retained tokens given in ascending position order, from the rule as printed:
    neighbours (i, i+g) become (i', i' + ln ln g), or (i', i' + g) while g <= 10; the first sits at 0."""
    out = [0.0]
    for a, b in zip(positions[:-1], positions[1:]):
        g = b - a
        out.append(out[-1] + (g if g <= 10 else math.log(math.log(g))))
    return out


def test_gap_function_on_worked_values():
    assert [compress_gap(g) for g in (1, 2, 10)] == [1.0, 2.0, 10.0]             # g <= 10 stays
    assert abs(compress_gap(11) - math.log(math.log(11))) < 1e-15                 # 0.8746...: the rule as printed
    # ln 986 = 6.893656, ln 6.893656 = 1.930602;  ln 70000 = 11.156251, ln 11.156251 = 2.412000
    assert abs(compress_gap(986) - 1.930602) < 1e-6 and abs(compress_gap(70000) - 2.412000) < 1e-6
    # positions (0, 3, 13, 14, 1000): gaps 3, 10, 1, 986
    assert np.allclose(chain([0, 3, 13, 14, 1000]), [0, 3, 13, 14, 14 + 1.930602], atol=1e-6)


def history_poscomp(q, k, v, positions, cap, scale, G):
    """TOVA with position compression over the full history: an order-preserving list of retained tokens;
    every step rotates the retained keys and the query afresh (complex form) at the chain's positions."""
    kept, res = [], []
    for t in range(q.shape[0]):
        kept.append(t)                                            # tokens arrive in position order
        cp = chain([positions[i] for i in kept])
        H = q.shape[1]
        out = np.zeros((H, q.shape[2]))
        w = np.zeros((H, len(kept)))
        for h in range(H):
            qr = rope_complex(q[t, h], cp[-1])
            kr = np.stack([rope_complex(k[i, h // G], cp[r]) for r, i in enumerate(kept)])
            w[h] = softmax64(scale * kr @ qr)
            out[h] = w[h] @ np.stack([v[i, h // G] for i in kept])
        if len(kept) > cap:
            del kept[int(np.argmin(w.mean(axis=0)))]
        res.append(({positions[i] for i in kept}, out, cp))
    return res


@pytest.mark.parametrize("H,Hkv,D,cap,T,stride", [(4, 4, 8, 6, 60, 1), (4, 2, 16, 10, 80, 7), (2, 1, 4, 5, 50, 37)])
def test_matches_history_restatement(H, Hkv, D, cap, T, stride):
    """stride > 1: tokens sit `stride` positions apart, so gaps above 10 arise at once."""
    q, k, v = random_stream(90 + cap, T, H, Hkv, D)
    positions = [3 + stride * t for t in range(T)]
    scale = 1.0 / np.sqrt(D)
    ref = history_poscomp(q, k, v, positions, cap, scale, H // Hkv)
    c = OracleCache(1, H, Hkv, D, cap, precision="f64", rope_base=BASE)
    saw_compression = False
    for t in range(T):
        out, *_ = c.step(q[t][None], k[t][None], v[t][None], positions[t])
        n = int(c.len[0])
        assert n == min(t + 1, cap)
        assert set(c.pos[0, :n].tolist()) == ref[t][0], t
        assert np.abs(out[0] - ref[t][1]).max() < 1e-10, t
        saw_compression |= max(np.diff(sorted(ref[t][0])), default=0) > 10
    assert saw_compression


def test_without_gaps_above_ten_it_is_ordinary_rotary_attention():
    """Capacity >= stream length and consecutive positions: nothing is dropped, every gap is 1, the new positions
    are the old ones (shifted to start at 0): causal attention over keys and queries rotated at their positions,
    by a library routine."""
    H, Hkv, D, T = 4, 2, 16, 40
    q, k, v = random_stream(17, T, H, Hkv, D)
    c = OracleCache(1, H, Hkv, D, T, precision="f64", rope_base=BASE)
    outs = np.stack([c.step(q[t][None], k[t][None], v[t][None], 100 + t)[0][0] for t in range(T)])   # [T,H,D]
    qr = np.stack([rope_complex(q[t], 100 + t) for t in range(T)])
    kr = np.stack([rope_complex(k[t], 100 + t) for t in range(T)])
    tq = torch.from_numpy(qr).permute(1, 0, 2)[None]
    tk = torch.from_numpy(kr).permute(1, 0, 2).repeat_interleave(H // Hkv, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(H // Hkv, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.abs(outs - ref).max() < 1e-10


def test_shifting_every_position_changes_nothing():
    H, Hkv, D, cap, T = 4, 4, 8, 7, 60
    q, k, v = random_stream(23, T, H, Hkv, D)
    a = OracleCache(1, H, Hkv, D, cap, precision="f64", rope_base=BASE)
    b = OracleCache(1, H, Hkv, D, cap, precision="f64", rope_base=BASE)
    for t in range(T):
        oa, ea, *_ = a.step(q[t][None], k[t][None], v[t][None], 13 * t)
        ob, eb, *_ = b.step(q[t][None], k[t][None], v[t][None], 13 * t + 50000)
        assert ea[0] == (eb[0] - 50000 if eb[0] >= 0 else -1)
        assert np.abs(oa - ob).max() < 1e-9
        assert np.abs(a.last_cpos - b.last_cpos).max() == 0


def test_compressed_positions_follow_the_chain_and_float_build_tracks_double():
    H, Hkv, D, cap, T = 4, 2, 16, 9, 70
    q, k, v = random_stream(29, T, H, Hkv, D)
    f = OracleCache(1, H, Hkv, D, cap, precision="f32", rope_base=BASE)
    d = OracleCache(1, H, Hkv, D, cap, precision="f64", rope_base=BASE)
    for t in range(T):
        n = int(d.len[0])
        held = d.pos[0, :n].tolist() + [11 * t]
        of, ef, *_ = f.step(q[t][None], k[t][None], v[t][None], 11 * t)
        od, ed, *_ = d.step(q[t][None], k[t][None], v[t][None], 11 * t)
        order = np.argsort(held)
        want = np.zeros(len(held))
        want[order] = chain(sorted(held))
        assert np.abs(d.last_cpos[0, :len(held)] - want).max() < 1e-12
        assert ef[0] == ed[0] and np.abs(of - od).max() < 5e-5
