"""One workspace, many kinds of calls in a shuffled order: every call is checked against the
oracle, so state that one entry point leaves behind in the workspace (counters, flags, staged
descriptors, candidates) cannot leak into the next one unnoticed."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device

pytestmark = pytest.mark.gpu


def test_shuffled_sequence_of_calls_on_one_workspace(ql):
    g = 128
    N_MAX = 9728
    ws = ql.new_workspace(64, N_MAX)
    rng = np.random.default_rng(20260)
    lin = {}
    for name, (K, N) in {"wide": (512, 9728), "tall": (2560, 1024), "mid": (1024, 2560), "head": (512, 4096)}.items():
        d = qsynth.make_linear([93, len(lin)], 64, K, N, g)
        lin[name] = (d, pack_on_device(ql, d), dev_u16(d["x"]))

    def want(name, M):
        d = lin[name][0]
        return orc.qlinear_f64(d["x"][:M], d["wq"], d["scale"], d["zero"], g)

    def single(name, M, path):
        d, p, x = lin[name]
        y = torch.full((M, d["N"]), 0x7FC0, dtype=torch.int16, device="cuda")
        ql.qlinear_w4a16(p, x[:M], y, None, M, d["K"], d["N"], g, ws, path=path)
        torch.cuda.synchronize()
        check_against_oracle(host_u16(y), want(name, M), f"single {name} M={M} path={path}")

    def single_tokens(name, M, path):
        d, p, x = lin[name]
        tok = torch.full((M,), -7, dtype=torch.int32, device="cuda")
        ql.qlinear_w4a16(p, x[:M], None, tok, M, d["K"], d["N"], g, ws, path=path)
        torch.cuda.synchronize()
        idx, gap = orc.argmax_rows(want(name, M))
        ok = gap >= 1e-3
        assert np.array_equal(tok.cpu().numpy().astype(np.int64)[ok], idx[ok]), f"tokens {name} M={M} path={path}"

    def stack_independent(names, M):
        ys = [torch.full((M, lin[n][0]["N"]), 0x7FC0, dtype=torch.int16, device="cuda") for n in names]
        ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=lin[n][0]["K"], N=lin[n][0]["N"], g=g, ld_in=lin[n][0]["K"],
                                ld_out=lin[n][0]["N"], packed=lin[n][1], in0=lin[n][2][:M], out=y) for n, y in zip(names, ys)])
        ql.qlinear_stack_w4a16(ops, ws)
        torch.cuda.synchronize()
        for n, y in zip(names, ys):
            check_against_oracle(host_u16(y), want(n, M), f"stack independent {n} M={M}")

    def stack_chain_with_tail(M):
        # wide (512 -> 9728 is not chainable into tall); use mid -> tall: 1024 -> 2560 -> 1024, then tokens and acceptance
        d1, p1, x1 = lin["mid"]
        d2, p2, _ = lin["tall"]
        y1 = torch.full((M, 2560), 0x7FC0, dtype=torch.int16, device="cuda")
        xn = torch.full((M, 2560), 0x7FC0, dtype=torch.int16, device="cuda")
        tok = torch.full((M,), -7, dtype=torch.int32, device="cuda")
        acc = torch.full((2,), -7, dtype=torch.int32, device="cuda")
        y1_64 = want("mid", M)
        ops = [dict(kind=ql.QL_OP_LINEAR, M=M, K=1024, N=2560, g=g, ld_in=1024, ld_out=2560, packed=p1, in0=x1[:M], out=y1),
               dict(kind=ql.QL_OP_UNIT_RMS, M=M, N=2560, ld_in=2560, ld_out=2560, in0=y1, out=xn)]
        # greedy tokens of the second linear on the GPU's own normalised input, then a draft that agrees on a prefix
        ql.qlinear_stack_w4a16(ql.make_ops(ops), ws)
        torch.cuda.synchronize()
        check_against_oracle(host_u16(y1), y1_64, f"chain first linear M={M}")
        y2_64 = orc.qlinear_f64(host_u16(xn), d2["wq"], d2["scale"], d2["zero"], g)
        idx, gap = orc.argmax_rows(y2_64)
        if not np.all(gap >= 1e-3):
            return
        a_plant = int(rng.integers(0, M + 1))
        draft = idx.copy()
        if a_plant < M:
            draft[a_plant] = (draft[a_plant] + 1) % 1024
        dr = torch.from_numpy(draft.astype(np.int32)).cuda()
        ops.append(dict(kind=ql.QL_OP_LINEAR, M=M, K=2560, N=1024, g=g, ld_in=2560, ld_out=1024, packed=p2, in0=xn, out=None,
                        argmax_out=tok, draft_ids=dr, accept_out=acc))
        ql.qlinear_stack_w4a16(ql.make_ops(ops), ws)
        torch.cuda.synchronize()
        assert np.array_equal(tok.cpu().numpy().astype(np.int64), idx), f"chain tokens M={M}"
        a, bonus = orc.accept_prefix(idx, draft)
        assert acc.cpu().numpy().tolist() == [a, bonus], f"chain acceptance M={M}"

    calls = [
        lambda: single("wide", 16, ql.QL_PATH_MMA), lambda: single("wide", 16, ql.QL_PATH_TC5), lambda: single("wide", 32, ql.QL_PATH_TC5),
        lambda: single("tall", 64, ql.QL_PATH_MMA), lambda: single("mid", 5, ql.QL_PATH_MMA), lambda: single("mid", 48, ql.QL_PATH_TC5),
        lambda: single_tokens("head", 16, ql.QL_PATH_MMA), lambda: single_tokens("head", 16, ql.QL_PATH_TC5),
        lambda: stack_independent(["wide", "tall", "mid"], 16), lambda: stack_independent(["tall", "mid"], 3),
        lambda: stack_independent(["wide", "head"], 16), lambda: stack_chain_with_tail(16), lambda: stack_chain_with_tail(7),
    ]
    order = rng.permutation(np.repeat(np.arange(len(calls)), 3))
    for i in order:
        calls[int(i)]()
        assert ql.ql_device_status(ws) == ql.QL_OK
