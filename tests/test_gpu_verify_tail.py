"""Verification tail on the device: the LM head's greedy tokens are compared with the drafted
tokens inside the kernel (accepted-prefix length and bonus token, no host round trip).  Checked bit
for bit against the oracle's accept_prefix on the oracle's own tokens, for planted agreement
prefixes of length 0, 1, 15 and 16 and a few in between, at the full vocabulary size and at a
small one with M < 16."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import dev_u16, pack_on_device

pytestmark = pytest.mark.gpu


def _run(ql, d, packed, ws, draft):
    M, K, N, g = d["M"], d["K"], d["N"], d["g"]
    tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    acc = torch.full((2,), -7, dtype=torch.int32, device="cuda")
    drf = torch.from_numpy(np.asarray(draft, dtype=np.int32)).cuda()
    ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=packed, in0=dev_u16(d["x"]),
                            out=None, argmax_out=tok, draft_ids=drf, accept_out=acc)])
    ql.qlinear_stack_w4a16(ops, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    return tok.cpu().numpy().astype(np.int64), tuple(int(v) for v in acc.cpu().numpy())


@pytest.mark.parametrize("M,N", [(16, qsynth.VOCAB), (5, 128 * 37)])
def test_accept_prefix_on_device(ql, M, N):
    d = qsynth.config3(N=N, M=M) if N == qsynth.VOCAB else qsynth.make_linear([61, M, N], M, 512, N, 128)
    packed = pack_on_device(ql, d)
    ws = ql.new_workspace(M, N)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], d["g"], col_block=8192)
    want_tok, gap = orc.argmax_rows(y64)
    assert gap.min() >= 1e-3, "a row of this seed has a near-tie; pick another seed"
    rng = np.random.default_rng(9)
    for a in sorted({0, 1, M // 2, M - 1, M}):
        draft = want_tok.copy()
        if a < M:
            draft[a] = (want_tok[a] + 1) % N                      # first disagreement at row a
            draft[a + 1:] = rng.integers(0, N, M - a - 1)
            if a + 2 < M:
                draft[a + 2] = want_tok[a + 2]                    # a later agreement does not count
        tok, acc = _run(ql, d, packed, ws, draft)
        assert np.array_equal(tok, want_tok)
        assert acc == orc.accept_prefix(want_tok, draft), (a, acc)
    # an entry of -1 never agrees
    draft = want_tok.copy()
    draft[M - 1] = -1
    _, acc = _run(ql, d, packed, ws, draft)
    assert acc == (M - 1, int(want_tok[M - 1]))
