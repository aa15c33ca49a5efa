"""Pins of the sliding-window attention oracle (CPU only): each test checks it against something
other than itself, chosen so that a plausible mistake - a one-sided window, an off-by-one edge, a
missing fallback, a wrong key/value head, a missing 1/sqrt(d) - fails one of them."""
import math

import numpy as np

from oracle import swa_oracle as so
from oracle import w4a16_oracle as orc


def bits(a):
    return orc.f64_to_bf16_bits(np.asarray(a, dtype=np.float64))


def test_key_range_from_the_definition():
    # Section 3.3: symmetric around the query, W div 2 on either side, clipped; full below the window
    assert so.swa_key_range(100, 1000, 8) == (96, 105)
    assert so.swa_key_range(2, 1000, 8) == (0, 7)
    assert so.swa_key_range(998, 1000, 8) == (994, 1000)
    assert so.swa_key_range(5, 8, 8) == (0, 8)            # fits into the window: everything
    assert so.swa_key_range(5, 9, 8) == (1, 9)            # one key too many: windowed
    assert so.swa_key_range(7, 64, 1024) == (0, 64)


def test_brute_force_pure_python():
    rng = np.random.default_rng(11)
    n_q, Hq, Hkv, d, T, W, p0 = 3, 4, 2, 4, 11, 4, 6
    qb, kb, vb = bits(rng.normal(size=(n_q, Hq, d))), bits(rng.normal(size=(T, Hkv, d))), bits(rng.normal(size=(T, Hkv, d)))
    q, k, v = orc.bf16_bits_to_f64(qb), orc.bf16_bits_to_f64(kb), orc.bf16_bits_to_f64(vb)
    got = so.swa_attention_f64(qb, kb, vb, p0, W)
    for i in range(n_q):
        p = p0 + i
        keys = [kk for kk in range(T) if abs(kk - p) <= W // 2]          # the sentence, written out
        for h in range(Hq):
            kvh = h // (Hq // Hkv)
            sc = [sum(q[i, h, c] * k[kk, kvh, c] for c in range(d)) / math.sqrt(d) for kk in keys]
            mx = max(sc)
            e = [math.exp(x - mx) for x in sc]
            z = sum(e)
            for c in range(d):
                want = sum(e[j] / z * v[kk, kvh, c] for j, kk in enumerate(keys))
                assert abs(got[i, h, c] - want) < 1e-12


def test_uniform_scores_give_the_mean_position_of_the_window():
    # keys all zero -> every visible key has weight 1/n; value = position -> output = mean position
    n_q, Hq, Hkv, d, T, W = 16, 2, 1, 8, 300, 64
    qb = bits(np.ones((n_q, Hq, d)))
    kb = bits(np.zeros((T, Hkv, d)))
    vb = bits(np.broadcast_to(np.arange(T, dtype=np.float64)[:, None, None], (T, Hkv, d)))   # positions above 256 round to even numbers: the expected mean uses the rounded values
    for p0 in (0, 20, 100, T - n_q):
        got = so.swa_attention_f64(qb, kb, vb, p0, W)
        for i in range(n_q):
            p = p0 + i
            lo, hi = max(0, p - 32), min(T - 1, p + 32)
            vals = orc.bf16_bits_to_f64(vb[lo:hi + 1, 0, 0])
            assert np.allclose(got[i], vals.mean(), rtol=0, atol=1e-9)
    # a query in the middle sees as many keys on its right as on its left
    sgn = bits(np.broadcast_to(np.sign(np.arange(T) - 150.0)[:, None, None], (T, Hkv, d)))
    got = so.swa_attention_f64(qb[:1], kb, sgn, 150, W)
    assert np.allclose(got, 0.0, atol=1e-12)


def test_full_attention_when_the_sequence_fits():
    n_q, Hq, Hkv, d, W = 4, 1, 1, 4, 64
    qb = bits(np.ones((n_q, Hq, d)))
    for T in (10, 64):
        kb = bits(np.zeros((T, Hkv, d)))
        vb = bits(np.broadcast_to(np.arange(T, dtype=np.float64)[:, None, None], (T, Hkv, d)))
        got = so.swa_attention_f64(qb, kb, vb, T - n_q, W)
        assert np.allclose(got, (T - 1) / 2.0, atol=1e-9)             # every key, for every query
    T = 65                                                              # one more key: the window applies
    kb = bits(np.zeros((T, Hkv, d)))
    vb = bits(np.broadcast_to(np.arange(T, dtype=np.float64)[:, None, None], (T, Hkv, d)))
    got = so.swa_attention_f64(qb, kb, vb, T - n_q, W)
    assert np.allclose(got[0], np.arange(T - n_q - 32, T).mean(), atol=1e-9)


def test_a_key_outside_the_window_cannot_leak_and_one_inside_dominates():
    n_q, Hq, Hkv, d, T, W, p0 = 1, 1, 1, 4, 200, 16, 100
    q = np.zeros((n_q, Hq, d)); q[0, 0, 0] = 8.0
    k = np.zeros((T, Hkv, d)); v = np.zeros((T, Hkv, d))
    k[p0 - 9, 0, 0] = 64.0; v[p0 - 9] = 1000.0           # just outside on the left (|k - p| = 9 > 8)
    k[p0 + 9, 0, 0] = 64.0; v[p0 + 9] = -1000.0          # just outside on the right
    got = so.swa_attention_f64(bits(q), bits(k), bits(v), p0, W)
    assert np.allclose(got, 0.0, atol=1e-12)
    k[p0 + 8, 0, 0] = 64.0; v[p0 + 8] = 7.0              # the last key inside, with an overwhelming score
    got = so.swa_attention_f64(bits(q), bits(k), bits(v), p0, W)
    assert np.allclose(got, 7.0, atol=1e-9)
    k[p0 + 8, 0, 0] = 0.0; k[p0 - 8, 0, 0] = 64.0; v[p0 - 8] = -3.0; v[p0 + 8] = 0.0
    got = so.swa_attention_f64(bits(q), bits(k), bits(v), p0, W)
    assert np.allclose(got, -3.0, atol=1e-9)


def test_scale_is_one_over_sqrt_d():
    # two visible keys with scores s and 0: the weights are sigmoid(s / sqrt(d)) and its complement
    d, T = 16, 2
    q = np.zeros((1, 1, d)); q[0, 0, 0] = 2.0
    k = np.zeros((T, 1, d)); k[0, 0, 0] = 3.0
    v = np.zeros((T, 1, d)); v[0] = 1.0
    got = so.swa_attention_f64(bits(q), bits(k), bits(v), 1, 8)
    want = 1.0 / (1.0 + math.exp(-(6.0 / 4.0)))
    assert np.allclose(got, want, atol=1e-12)


def test_softmax_shift_invariance_and_head_mapping():
    rng = np.random.default_rng(5)
    n_q, Hq, Hkv, d, T, W, p0 = 5, 8, 2, 8, 90, 20, 60
    qb, vb = bits(rng.normal(size=(n_q, Hq, d))), bits(rng.normal(size=(T, Hkv, d)))
    kb = bits(rng.integers(-16, 17, size=(T, Hkv, d)) / 8.0)             # multiples of 1/8: a shift by 2 stays exact in bf16
    base = so.swa_attention_f64(qb, kb, vb, p0, W)
    # adding one vector to every key adds q.c to every score of a query: the weights do not change
    c = np.zeros((1, 1, d)); c[0, 0, :] = 2.0
    kshift = bits(orc.bf16_bits_to_f64(kb) + c)
    assert np.array_equal(orc.bf16_bits_to_f64(kshift), orc.bf16_bits_to_f64(kb) + c)
    got = so.swa_attention_f64(qb, kshift, vb, p0, W)
    assert np.allclose(got, base, atol=1e-9)
    # value = index of the key/value head: query head h must read head h div 4
    vh = bits(np.broadcast_to(np.arange(Hkv, dtype=np.float64)[None, :, None], (T, Hkv, d)))
    got = so.swa_attention_f64(qb, kb, vh, p0, W)
    for h in range(Hq):
        assert np.allclose(got[:, h, :], h // 4, atol=1e-12)
