"""CPU oracle for the drafter's symmetric sliding-window attention.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu-baseline legs may import this file; the
product path never does, and this file imports nothing from the product.

What it computes.  The paper's drafter attends bidirectionally from the mask-token queries of the
drafted block and, to bound the cost on long contexts, restricts every query to a fixed-size
window that is symmetric around the query - not a causal, left-only one (Section 3.3, "Drafter
SWA": windows of 1,024 or 2,048 tokens; Section 2.3).  The restriction is applied inside the
attention computation only: the key/value cache stays complete, nothing is evicted or rotated.
Sequences that fit into the window are attended in full.  The paper prints no formula; the
definition below is the plain one, and the points it leaves open are fixed as follows:

  * window.  A query at position p sees the keys k with |k - p| <= W div 2 (W div 2 positions on
    either side and its own), clipped to the cache [0, T).  If T <= W, every query sees every key.
  * queries.  The n_q queries of a block stand at consecutive positions p0, p0 + 1, ...
  * attention.  out[i, h, :] = sum_k softmax_k(q[i, h, :] . key[k, h div (Hq div Hkv), :] / sqrt(d))
    * value[k, h div (Hq div Hkv), :]   (grouped-query attention: Hq div Hkv query heads share
    one key/value head), softmax over the visible keys only; q, key, value are bf16, all
    arithmetic here is fp64.  Positional rotation, if any, has been applied to q and key before.

Every function is pinned by tests/test_swa_oracle_pins.py to something other than itself: a
pure-Python brute force with the key set written from the sentence above, closed forms (uniform
scores: the output is the mean of the visible values), a value that must not leak from just
outside the window, and the shift invariance of the softmax.
"""
from __future__ import annotations

import numpy as np


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def swa_key_range(p: int, T: int, window: int):
    """First and one-past-last key a query at position p sees in a cache of T keys (Section 3.3:
    symmetric window around the query; full attention when the sequence fits into the window)."""
    if T <= window:
        return 0, T
    half = window // 2
    return max(0, p - half), min(T, p + half + 1)


def swa_attention_f64(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, p0: int, window: int) -> np.ndarray:
    """q_bits [n_q, Hq, d], k_bits / v_bits [T, Hkv, d] (bf16 bit patterns) -> out float64 [n_q, Hq, d]."""
    q = _bf16_to_f64(q_bits)
    k = _bf16_to_f64(k_bits)
    v = _bf16_to_f64(v_bits)
    n_q, Hq, d = q.shape
    T, Hkv, _ = k.shape
    assert Hq % Hkv == 0 and v.shape == k.shape and k.shape[2] == d
    group = Hq // Hkv
    out = np.zeros((n_q, Hq, d), dtype=np.float64)
    for i in range(n_q):
        lo, hi = swa_key_range(p0 + i, T, window)
        for h in range(Hq):
            kv = h // group
            s = k[lo:hi, kv, :] @ q[i, h, :] / np.sqrt(float(d))          # [hi - lo]
            w = np.exp(s - s.max())
            w /= w.sum()
            out[i, h, :] = w @ v[lo:hi, kv, :]
    return out
