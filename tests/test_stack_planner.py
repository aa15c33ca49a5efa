"""Host logic of the stack launcher, without a GPU: which operations are fused into the persistent
kernel, which gate/up pairs become dual operations, which glue operations are folded, which runs
are independent linears streamed as one piece per thread block, and what falls back to single launches.
Pointers are fake (never dereferenced: ql_stack_plan launches nothing)."""
import pytest

import qsynth


@pytest.fixture(scope="module")
def ql():
    from paper_2607_04244_b200 import build
    build.build_library()
    import paper_2607_04244_b200 as p
    p.load()
    return p


P = 0x1000000


def buf(i):
    return P + i * 0x1000000


def layer_ops(l, M=16, g=128, S=qsynth.LAYER_SHAPES):
    L, U, SU = 0, 1, 2
    h_in, h_out = buf(1 + (l % 2)), buf(1 + ((l + 1) % 2))

    def lin(nm, x, ldx, y):
        return dict(kind=L, M=M, K=S[nm][0], N=S[nm][1], g=g, ld_in=ldx, ld_out=S[nm][1],
                    packed=buf(100 + 5 * l + list(S).index(nm)), in0=x, out=y)

    return [lin("qkv", h_in, 2560, buf(3)), dict(kind=U, M=M, N=4096, ld_in=6144, ld_out=4096, in0=buf(3), out=buf(4)),
            lin("o", buf(4), 4096, buf(5)), dict(kind=U, M=M, N=2560, ld_in=2560, ld_out=2560, in0=buf(5), out=buf(6)),
            lin("gate", buf(6), 2560, buf(7)), lin("up", buf(6), 2560, buf(8)),
            dict(kind=SU, M=M, N=9728, ld_in=9728, ld_out=9728, in0=buf(7), in1=buf(8), out=buf(9)),
            lin("down", buf(9), 9728, buf(10)), dict(kind=U, M=M, N=2560, ld_in=2560, ld_out=2560, in0=buf(10), out=h_out)]


def plan(ql, ops, M=16, N=151936):
    return ql.ql_stack_plan(ql.make_ops(ops), P, ql.ql_workspace_bytes(M, N))


def test_verify_step_is_one_launch(ql):
    ops = [o for l in range(36) for o in layer_ops(l)]
    ops.append(dict(kind=0, M=16, K=2560, N=151936, g=128, ld_in=2560, ld_out=151936, packed=buf(99), in0=buf(1),
                    out=None, argmax_out=buf(11)))
    c = plan(ql, ops)
    # 4 fused operations per layer (qkv, o, gate+up, down) + the LM head; every glue operation folded
    assert c == dict(stack_launches=1, fused_ops=145, dual_ops=36, folded_glue=144, independent=0,
                     single_linears=0, single_glue=0, batch_launches=0)


def test_trailing_glue_runs_on_its_own(ql):
    c = plan(ql, layer_ops(0))
    assert c["stack_launches"] == 1 and c["fused_ops"] == 4 and c["folded_glue"] == 3 and c["single_glue"] == 1


def test_gate_up_without_their_glue_stay_two_operations(ql):
    ops = layer_ops(0)[4:6]                      # gate, up only
    c = plan(ql, ops)
    assert c["fused_ops"] == 2 and c["dual_ops"] == 0
    # up shares no buffer with gate except the input both read: the two run as one stream of chunks
    assert c["independent"] == 1 and c["batch_launches"] == 1


def test_independent_linears_skip_the_wait_but_write_after_write_does_not(ql):
    def lin(i, out):
        return dict(kind=0, M=16, K=2560, N=9728, g=128, ld_in=2560, ld_out=9728, packed=buf(100 + i), in0=buf(1), out=out)
    c = plan(ql, [lin(i, buf(20 + i)) for i in range(6)])
    assert c["fused_ops"] == 6 and c["independent"] == 5 and c["batch_launches"] == 1
    c = plan(ql, [lin(i, buf(20)) for i in range(6)])          # same output buffer: ordered
    assert c["independent"] == 0 and c["batch_launches"] == 0
    # independent of the neighbour but not pairwise (ops 0 and 2 write the same buffer): a chain
    c = plan(ql, [lin(0, buf(20)), lin(1, buf(21)), lin(2, buf(20))])
    assert c["independent"] == 0 and c["batch_launches"] == 0
    # any K runs as one stream: the X operand comes chunk by chunk through a ring of slots
    def wide(i):
        return dict(kind=0, M=16, K=9728, N=2560, g=128, ld_in=9728, ld_out=2560, packed=buf(100 + i), in0=buf(1), out=buf(20 + i))
    c = plan(ql, [wide(i) for i in range(40)])
    assert c["fused_ops"] == 40 and c["batch_launches"] == 1 and c["independent"] == 39
    # a linear that reads its predecessor's output is dependent
    a = dict(kind=0, M=16, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100), in0=buf(1), out=buf(2))
    b = dict(kind=0, M=16, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(101), in0=buf(2), out=buf(3))
    assert plan(ql, [a, b])["independent"] == 0


def test_lists_of_plain_linears_above_16_rows_become_slabs(ql):
    def big(i, M, out=None):
        return dict(kind=0, M=M, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100 + i), in0=buf(1), out=buf(20 + i) if out is None else out)
    c = plan(ql, [big(i, 64) for i in range(3)], M=64)
    assert c["stack_launches"] == 1 and c["fused_ops"] == 12 and c["batch_launches"] == 1 and c["single_linears"] == 0
    c = plan(ql, [big(i, 40) for i in range(2)], M=64)
    assert c["fused_ops"] == 6 and c["batch_launches"] == 1                      # 16 + 16 + 8 rows
    c = plan(ql, [big(0, 32), big(1, 48)], M=64)                                  # different row counts: one launch each
    assert c["stack_launches"] == 0 and c["single_linears"] == 2
    c = plan(ql, [big(0, 32, out=buf(20)), big(1, 32, out=buf(20))], M=64)        # same output: ordered, one launch each
    assert c["stack_launches"] == 0 and c["single_linears"] == 2


def test_m_above_16_and_mixed_group_sizes(ql):
    big = dict(kind=0, M=32, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100), in0=buf(1), out=buf(2))
    c = plan(ql, [big, big], M=32)
    assert c["stack_launches"] == 0 and c["single_linears"] == 2
    a = dict(kind=0, M=16, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100), in0=buf(1), out=buf(2))
    b = dict(a, g=64, in0=buf(2), out=buf(3), packed=buf(101))
    c = plan(ql, [a, b])
    assert c["stack_launches"] == 2 and c["fused_ops"] == 2     # one launch per group size


def test_unmatched_glue_is_not_folded(ql):
    a = dict(kind=0, M=16, K=2560, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100), in0=buf(1), out=buf(2))
    stray = dict(kind=1, M=16, N=2560, ld_in=2560, ld_out=2560, in0=buf(7), out=buf(8))     # not a's output
    b = dict(a, in0=buf(8), out=buf(3), packed=buf(101))
    c = plan(ql, [a, stray, b])
    assert c["folded_glue"] == 0 and c["single_glue"] == 1 and c["fused_ops"] == 2 and c["stack_launches"] == 2
    # a glue whose output is NOT what the next linear reads is launched on its own as well
    g1 = dict(kind=1, M=16, N=2560, ld_in=2560, ld_out=2560, in0=buf(2), out=buf(9))
    c = plan(ql, [a, g1, b])
    assert c["folded_glue"] == 0 and c["single_glue"] == 1


def test_plan_validates_like_the_launcher(ql):
    bad = dict(kind=0, M=16, K=100, N=2560, g=128, ld_in=2560, ld_out=2560, packed=buf(100), in0=buf(1), out=buf(2))
    with pytest.raises(ql.QlError) as e:
        plan(ql, [bad])
    assert e.value.status == ql.QL_ERR_SHAPE


def test_stream_k_split_is_balanced_contiguous_and_invertible(ql):
    """CTA i owns chunks [first(i), first(i+1)); the ranges tile [0, total), differ by at most one
    chunk in length, and the owner lookup (float guess + exact correction on the device) inverts them."""
    lib = ql.load()
    import random
    rnd = random.Random(7)
    cases = [(1520, 148), (640, 148), (960, 148), (23740, 148), (8, 148), (1, 148), (148, 148), (149, 148), (3040, 148)]
    cases += [(rnd.randint(1, 40000), rnd.randint(1, 160)) for _ in range(60)]
    for total, ncta in cases:
        nc = min(ncta, total)
        firsts = [lib.ql_plan_first_chunk(total, ncta, i) for i in range(nc + 1)]
        assert firsts[0] == 0 and firsts[-1] == total
        sizes = [b - a for a, b in zip(firsts, firsts[1:])]
        assert min(sizes) >= 1 and max(sizes) - min(sizes) <= 1
        assert firsts == [(i * total) // nc for i in range(nc + 1)]      # the 64-bit definition
        probes = {0, total - 1} | {rnd.randrange(total) for _ in range(40)} | set(firsts[:-1]) | {f - 1 for f in firsts[1:]}
        for c in probes:
            o = lib.ql_plan_chunk_owner(total, ncta, c)
            assert firsts[o] <= c < firsts[o + 1], (total, ncta, c, o)


def test_chain_split_aligned_where_tiles_can_have_thread_blocks_of_their_own(ql):
    """Chained operations: with at most ncta / 2 tiles and two chunks per thread block the aligned
    split is taken - pieces tile [0, total), no piece crosses a tile boundary, the thread blocks of
    a tile are consecutive, the first of them (the owner) has the extra chunks, and `last_cta` is
    the last thread block of the piece's tile.  Otherwise the even split, as before."""
    import random
    rnd = random.Random(11)
    try:
        for extra in (-1, 0, 3, 7, 500, -2):
            ql.ql_debug_set_owner_extra(extra)
            cases = [(20, 32, 148), (20, 76, 148), (48, 20, 148), (76, 20, 148), (1187, 20, 148), (20, 3, 148), (74, 4, 148),
                     (74, 3, 148), (1, 40, 148), (1, 400, 148), (3, 1000, 160), (20, 64, 132)]
            cases += [(rnd.randint(1, 90), rnd.randint(1, 160), rnd.randint(2, 160)) for _ in range(40)]
            for nt, gn, ncta in cases:
                rs = [ql.ql_plan_chain_split(nt, gn, ncta, i) for i in range(ncta)]
                total, pos = nt * gn, 0
                for r in rs:
                    if r["lo"] < r["hi"]:
                        assert r["lo"] == pos
                        pos = r["hi"]
                assert pos == total, (nt, gn, ncta, extra)
                most = -(-ncta // nt)
                want_aligned = extra >= -1 and 2 * nt <= ncta and gn >= 2 * most
                assert all(r["aligned"] == want_aligned for r in rs)
                if not want_aligned:
                    nc = min(ncta, total)
                    assert [r["lo"] for r in rs[:nc]] == [(i * total) // nc for i in range(nc)]
                    continue
                e = 0 if extra == -1 else extra
                for T in range(nt):
                    ctas = [i for i, r in enumerate(rs) if r["lo"] // gn == T]
                    assert ctas == list(range(ctas[0], ctas[-1] + 1)) and len(ctas) >= 2
                    assert ctas[0] == (T * ncta) // nt and ctas[-1] + 1 == ((T + 1) * ncta) // nt
                    sizes = [rs[i]["hi"] - rs[i]["lo"] for i in ctas]
                    assert all((rs[i]["hi"] - 1) // gn == T and rs[i]["last_cta"] == ctas[-1] for i in ctas)
                    assert min(sizes) >= 1 and sum(sizes) == gn
                    e_eff = min(e, gn - most)
                    rest = sizes[1:]
                    assert max(rest) - min(rest) <= 1
                    assert sizes[0] == e_eff + (gn - e_eff) // len(ctas)
    finally:
        ql.ql_debug_set_owner_extra(-1)


def test_verification_tail_argument_errors(ql):
    P = 0x100000
    base = dict(kind=ql.QL_OP_LINEAR, M=16, K=512, N=256, g=128, ld_in=512, ld_out=256, packed=P, in0=P, out=P)
    wsb = ql.ql_workspace_bytes(64, 256)

    def status(**kw):
        arr = ql.make_ops([dict(base, **kw)])
        try:
            ql.ql_stack_plan(arr, P, wsb)
            return ql.QL_OK
        except ql.QlError as e:
            return e.status
    assert status(argmax_out=P, draft_ids=P, accept_out=P) == ql.QL_OK
    assert status(argmax_out=P, draft_ids=P) == ql.QL_ERR_NULL            # accept_out missing
    assert status(draft_ids=P, accept_out=P) == ql.QL_ERR_NULL            # needs the arg-max
    assert status(argmax_out=P, draft_ids=P + 2, accept_out=P) == ql.QL_ERR_ALIGN
    assert status(M=32, argmax_out=P, draft_ids=P, accept_out=P) == ql.QL_ERR_UNSUPPORTED
