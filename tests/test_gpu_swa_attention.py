"""GPU parity of qattn_swa_bf16 (the drafter's symmetric sliding-window attention, paper Section
3.3) against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import swa_oracle as so
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16

pytestmark = pytest.mark.gpu


def run_case(ql, n_q, T, Hq, Hkv, p0, window, seed, ws=None, pad=0):
    d = 128
    q, k, v = qsynth.attention_inputs(seed, n_q, T, Hq, Hkv, d)
    ld_q, ld_kv = Hq * d + pad, Hkv * d + pad
    Q = torch.zeros((n_q, ld_q), dtype=torch.int16, device="cuda")
    K = torch.zeros((T, ld_kv), dtype=torch.int16, device="cuda")
    V = torch.zeros((T, ld_kv), dtype=torch.int16, device="cuda")
    Q[:, :Hq * d] = dev_u16(q.reshape(n_q, Hq * d))
    K[:, :Hkv * d] = dev_u16(k.reshape(T, Hkv * d))
    V[:, :Hkv * d] = dev_u16(v.reshape(T, Hkv * d))
    out = torch.full((n_q, ld_q), 0x7FC0, dtype=torch.int16, device="cuda")      # NaN-prefilled
    if ws is None:
        ws = ql.new_attn_workspace(Hq, Hkv)
    ql.qattn_swa_bf16(Q, K, V, out, n_q, T, Hq, Hkv, d, p0, window, ws, ld_q=ld_q, ld_kv=ld_kv, ld_out=ld_q)
    torch.cuda.synchronize()
    got = host_u16(out)
    want = so.swa_attention_f64(q, k, v, p0, window)
    check_against_oracle(got[:, :Hq * d], want.reshape(n_q, Hq * d), f"swa n_q={n_q} T={T} W={window} p0={p0}")
    if pad:
        assert np.all(got[:, Hq * d:] == 0x7FC0), "padding columns were written"
    return got, ws


# the paper's contexts (Section 3.4: 64, 2048 and 8192 input tokens) with the block appended, windows 1024 / 2048
@pytest.mark.parametrize("ctx,window", [(64, 1024), (2048, 1024), (2048, 2048), (8192, 1024), (8192, 2048)])
def test_paper_contexts_block_at_the_end(ql, ctx, window):
    T = ctx + 16
    run_case(ql, 16, T, 32, 8, T - 16, window, seed=ctx + window)


def test_block_in_the_middle_sees_both_sides(ql):
    # symmetric window: keys after the block are visible too
    T, window = 4096, 1024
    plan = ql.ql_attn_plan(16, T, 32, 8, 128, 2000, window)
    assert plan["key_lo"] == 2000 - 512 and plan["key_hi"] == 2015 + 512 + 1
    run_case(ql, 16, T, 32, 8, 2000, window, seed=7)


def test_block_at_the_start_and_clipped_windows(ql):
    run_case(ql, 16, 3000, 32, 8, 0, 1024, seed=8)
    run_case(ql, 16, 3000, 32, 8, 100, 1024, seed=9)


@pytest.mark.parametrize("n_q,T,Hq,Hkv,p0,window", [
    (5, 200, 8, 2, 150, 6),          # tiny window: most of a sub-block is masked, rows differ in what they see
    (16, 333, 8, 8, 300, 64),        # no grouping (one query head per key/value head), ragged last sub-block
    (1, 77, 16, 2, 76, 0),           # a window of zero: the query sees itself only
    (16, 64, 16, 8, 48, 64),         # T == window: full attention
    (16, 65, 16, 8, 49, 64),         # one key more: the window applies
    (7, 5000, 4, 4, 2500, 4000),     # window larger than what one piece per SM holds in one sub-block
])
def test_odd_shapes(ql, n_q, T, Hq, Hkv, p0, window):
    run_case(ql, n_q, T, Hq, Hkv, p0, window, seed=n_q * 1000 + T, pad=8)


def test_window_of_zero_returns_the_value_row(ql):
    d, T, Hq, Hkv = 128, 40, 4, 2
    q, k, v = qsynth.attention_inputs(3, 3, T, Hq, Hkv, d)
    got, _ = run_case(ql, 3, T, Hq, Hkv, 10, 0, seed=3)
    for i in range(3):
        for h in range(Hq):
            assert np.array_equal(got[i, h * d:(h + 1) * d], v[10 + i, h // 2, :])      # softmax over one key: exactly the value


def test_runs_are_bit_identical_and_workspace_is_reusable(ql):
    a, ws = run_case(ql, 16, 2064, 32, 8, 2048, 1024, seed=21)
    b, _ = run_case(ql, 16, 2064, 32, 8, 2048, 1024, seed=21, ws=ws)
    assert np.array_equal(a, b)
    run_case(ql, 16, 8208, 32, 8, 8192, 2048, seed=22, ws=ws)


def test_argument_errors(ql):
    d = 128
    ws = ql.new_attn_workspace(32, 8)
    z = lambda *s: torch.zeros(s, dtype=torch.int16, device="cuda")
    Q, K, V, out = z(16, 32 * d), z(100, 8 * d), z(100, 8 * d), z(16, 32 * d)
    with pytest.raises(ql.QlError) as e:
        ql.qattn_swa_bf16(Q, K, V, out, 16, 100, 32, 8, d, 90, 64, ws)          # the block sticks out of the cache
    assert e.value.status == ql.QL_ERR_SHAPE
    with pytest.raises(ql.QlError) as e:
        ql.qattn_swa_bf16(Q, K, V, out, 16, 100, 32, 8, 64, 0, 64, ws)          # head size
    assert e.value.status == ql.QL_ERR_UNSUPPORTED
    with pytest.raises(ql.QlError) as e:
        ql.qattn_swa_bf16(Q, K, V, out, 17, 100, 32, 8, d, 0, 64, ws)
    assert e.value.status == ql.QL_ERR_SHAPE
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(ql.QlError) as e:
        ql.qattn_swa_bf16(Q, K, V, out, 16, 100, 32, 8, d, 0, 64, small)
    assert e.value.status == ql.QL_ERR_WORKSPACE
