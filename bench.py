#!/usr/bin/env python
"""Benchmark of the W4A16 verify-step linears on B200.

Default workload ("verify_step"): one verify step of a 4B-class decoder at M=16 drafted tokens,
W4A16 with groups of 128 - the 36-layer linear stack (fused qkv, o, gate, up, down per layer,
chained through the unit-RMS glue) followed by the LM head with its arg-max - run through
qlinear_stack_w4a16.  One step streams every packed weight once (2.15 GB > L2, so every step is
cold).  value = algorithmic HBM bytes of the step / time, in GB/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sweep]

N > 1 (under torchrun): every rank runs an independent replica of the step on its own GPU
(the path has no exchange step); value is the aggregate over ranks, time is the max over ranks.
--impl reference times the CPU oracle on a bounded sample of the same workload.
--sweep prints one JSON line per point of the M-sweep (M x shape x group size x zero mode).
--swa prints the drafter's sliding-window attention points only.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import qsynth  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of the dominant kernel from an ncu capture of a 3-layer launch of the stack kernel:
# dram read + write = 161.91 MB for 162.32 MB of algorithmic bytes.  Traffic grows in proportion to the
# layers streamed (every packed byte crosses HBM once), so a full launch is scaled by this ratio.
NCU_TRAFFIC_RATIO = 161.91 / 162.32


# ------------------------------------------------------------------------------------------------
# byte accounting (algorithmic bytes: packed codes + bf16 scales + 4-bit zeros + bf16 X + bf16 Y)

def linear_bytes(M, K, N, g, y_bytes=True):
    return K * N // 2 + (K // g) * N * 2 + (K // g) * N // 2 + 2 * M * K + (2 * M * N if y_bytes else 0)


def step_bytes(M=16, g=128, n_layers=qsynth.N_LAYERS, lm_head=True):
    per_layer = sum(linear_bytes(M, K, N, g) for (K, N) in qsynth.LAYER_SHAPES.values())
    total = n_layers * per_layer
    if lm_head:
        total += linear_bytes(M, qsynth.HIDDEN, qsynth.VOCAB, g, y_bytes=False) + 4 * M   # tokens only
    return total, per_layer


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks during the timed region

class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.rows, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for (_, r) in self.rows]
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except Exception:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# the model on the device

def device_linear(ql, torch, seed, K, N, g, symmetric=False):
    """Seeded synthetic weights drawn ON THE DEVICE (same distributions as qsynth.make_linear,
    torch's generator instead of numpy's) and repacked with qpack_w4_g128."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    wq = torch.randint(-2 ** 31, 2 ** 31 - 1, (K // 8, N), dtype=torch.int32, device="cuda", generator=gen)
    sc = (torch.randn((K // g, N), device="cuda", generator=gen).abs() * 0.01 + 1e-3).to(torch.bfloat16).view(torch.int16)
    zero = None if symmetric else torch.randint(0, 16, (K // g, N), dtype=torch.uint8, device="cuda", generator=gen)
    return ql.qpack_w4_g128(wq, sc, zero, K, N, g)


class VerifyStep:
    """Packed weights, activation buffers and the operation list of one verify step."""

    def __init__(self, ql, torch, M=16, g=128, n_layers=qsynth.N_LAYERS, lm_head=True, symmetric=False):
        self.ql, self.torch, self.M, self.g, self.n_layers = ql, torch, M, g, n_layers
        S = qsynth.LAYER_SHAPES
        hid, mlp, qd = qsynth.HIDDEN, qsynth.MLP_DIM, qsynth.Q_DIM
        z = lambda w: torch.zeros((M, w), dtype=torch.int16, device="cuda")
        self.h = [z(hid), z(hid)]
        self.h_in = z(hid)
        b = dict(qkv=z(S["qkv"][1]), a=z(qd), o=z(hid), r=z(hid), gt=z(mlp), up=z(mlp), d=z(mlp), dn=z(hid))
        self.tokens = torch.zeros((M,), dtype=torch.int32, device="cuda")
        L, U, SU = ql.QL_OP_LINEAR, ql.QL_OP_UNIT_RMS, ql.QL_OP_SILU_MUL_UNIT_RMS
        self.packed, ops = [], []
        for l in range(n_layers):
            pk = {nm: device_linear(ql, torch, 1000 * l + i, S[nm][0], S[nm][1], g, symmetric) for i, nm in enumerate(S)}
            self.packed.append(pk)
            src = self.h_in if l == 0 else self.h[(l - 1) % 2]
            dst = self.h[l % 2]

            def lin(nm, x, y):
                return dict(kind=L, M=M, K=S[nm][0], N=S[nm][1], g=g, ld_in=x.shape[1], ld_out=y.shape[1],
                            packed=pk[nm], in0=x, out=y)

            def glue(kind, a, b2, out, N):
                return dict(kind=kind, M=M, N=N, ld_in=a.shape[1], ld_out=out.shape[1], in0=a, in1=b2, out=out)

            ops += [lin("qkv", src, b["qkv"]), glue(U, b["qkv"], None, b["a"], qd), lin("o", b["a"], b["o"]),
                    glue(U, b["o"], None, b["r"], hid), lin("gate", b["r"], b["gt"]), lin("up", b["r"], b["up"]),
                    glue(SU, b["gt"], b["up"], b["d"], mlp), lin("down", b["d"], b["dn"]),
                    glue(U, b["dn"], None, dst, hid)]
        self.h_last = self.h[(n_layers - 1) % 2]
        self.lm = None
        if lm_head:
            self.lm = device_linear(ql, torch, 999983, hid, qsynth.VOCAB, g)
            ops.append(dict(kind=L, M=M, K=hid, N=qsynth.VOCAB, g=g, ld_in=hid, ld_out=qsynth.VOCAB, packed=self.lm,
                            in0=self.h_last, out=None, argmax_out=self.tokens))
        self.bufs = b
        self.op_dicts = ops
        self.ops = ql.make_ops(ops)
        self.linear_ops = ql.make_ops([o for o in ops if o["kind"] == L])
        self.n_linear = len(self.linear_ops)
        self.ws = ql.new_workspace(M, qsynth.VOCAB if lm_head else mlp)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(4242)
        self.h_in.copy_(torch.randn((M, hid), device="cuda", generator=gen).to(torch.bfloat16).view(torch.int16))
        self.host_in = self.h_in.cpu().pin_memory()
        self.host_tokens = torch.zeros((M,), dtype=torch.int32).pin_memory()

    def run(self):
        self.ql.qlinear_stack_w4a16(self.ops, self.ws)

    def run_linears_only(self):
        self.ql.qlinear_stack_w4a16(self.linear_ops, self.ws)

    def run_host(self):
        self.ql.qlinear_stack_w4a16_host(self.ops, self.host_in, self.h_in, self.tokens, self.host_tokens, self.ws)


def independent_point(ql, torch, M, K, N, g, packed, ws, sym=False, iters=5):
    """Throughput of one linear shape with cold L2: the distinct weight sets `packed` (together more
    than twice the L2), one input, DISTINCT outputs, back to back: the whole list is one
    qlinear_stack_w4a16 call (independent operations: nothing waits for a result; above 16 rows the
    launcher cuts every linear into slabs of 16 rows).  Returns microseconds per linear and the kernel."""
    R = len(packed)
    xin = torch.randn((M, K), device="cuda").to(torch.bfloat16).view(torch.int16)
    youts = [torch.zeros((M, N), dtype=torch.int16, device="cuda") for _ in range(R)]
    ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=p, in0=xin, out=y)
                       for p, y in zip(packed, youts)])
    plan = ql.ql_stack_plan(ops, ws.data_ptr(), ws.numel())
    fn = lambda: ql.qlinear_stack_w4a16(ops, ws)
    if plan["batch_launches"] == plan["stack_launches"] == 1 and plan["single_linears"] == 0:
        kernel = "qstack_tc5_kernel, one stream of chunks" + ("" if M <= 16 else f", {(M + 15) // 16} slabs of 16 rows per linear")
    else:
        kernel = f"planner: {plan}"
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    ts = sorted(time_events(torch, fn, 1) / R * 1e3 for _ in range(iters))
    us = ts[len(ts) // 2]
    b = linear_bytes(M, K, N, g) - ((K // g) * N // 2 if sym else 0)
    peak, _ = measured_peak()
    return {"M": M, "K": K, "N": N, "g": g, "zero": "sym8" if sym else "asym", "us": us, "us_min": ts[0], "bytes": b,
            "GBps": b / us / 1e3, "frac_of_measured_peak": b / us / 1e3 / peak, "frac_of_8TBs": b / us / 1e3 / NOMINAL_HBM_GBS,
            "kernel": kernel, "weight_sets": R}


def swa_points(ql, torch, caches=32, iters=5):
    """The drafter's sliding-window attention (paper Section 3.3) at the paper's three input lengths and its
    two windows, plus full attention at the long length: `caches` distinct key/value caches back to
    back (together more than twice the L2 wherever a call reads more than a few MB), one call each,
    time / caches.  Bytes = the keys and values inside the union of the 16 queries' windows + Q + out."""
    Hq, Hkv, d, n_q = qsynth.ATTN_HEADS, qsynth.ATTN_KV_HEADS, qsynth.ATTN_HEAD_DIM, 16
    ws = ql.new_attn_workspace(Hq, Hkv)
    peak, _ = measured_peak()
    rows = []
    for ctx in qsynth.SWA_CONTEXTS:
        T = ctx + n_q
        K = [torch.randn((T, Hkv * d), device="cuda").to(torch.bfloat16).view(torch.int16) for _ in range(caches)]
        V = [torch.randn((T, Hkv * d), device="cuda").to(torch.bfloat16).view(torch.int16) for _ in range(caches)]
        Q = torch.randn((n_q, Hq * d), device="cuda").to(torch.bfloat16).view(torch.int16)
        outs = [torch.zeros((n_q, Hq * d), dtype=torch.int16, device="cuda") for _ in range(caches)]
        for window in qsynth.SWA_WINDOWS + ((1 << 20,) if ctx == qsynth.SWA_CONTEXTS[-1] else ()):
            plan = ql.ql_attn_plan(n_q, T, Hq, Hkv, d, ctx, window)

            def fn():
                for k, v, o in zip(K, V, outs):
                    ql.qattn_swa_bf16(Q, k, v, o, n_q, T, Hq, Hkv, d, ctx, window, ws)
            for _ in range(2):
                fn()
            torch.cuda.synchronize()
            # a call takes less device time than the host needs to enqueue it through the binding: the
            # stream is held back by a spin kernel while the calls are enqueued, so that the events
            # bracket device time only
            def timed():
                a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda._sleep(6_000_000)
                a.record()
                fn()
                e.record()
                e.synchronize()
                return a.elapsed_time(e)
            ts = sorted(timed() / caches * 1e3 for _ in range(iters))
            us = ts[len(ts) // 2]
            b = 2 * (plan["key_hi"] - plan["key_lo"]) * Hkv * d * 2 + 2 * n_q * Hq * d * 2
            rows.append({"context": ctx, "window": "full" if window >= T else window, "keys_read": plan["key_hi"] - plan["key_lo"],
                         "thread_blocks": plan["n_pieces"] * Hkv, "us": us, "us_min": ts[0], "bytes": b, "GBps": b / us / 1e3,
                         "frac_of_measured_peak": b / us / 1e3 / peak, "kernel": "qattn_swa_kernel, one launch per call"})
        del K, V, outs
        torch.cuda.empty_cache()
    return rows


def max_over_ranks(x: float, world: int, device="cuda") -> float:
    """The slowest rank's time (every rank runs its own replica; the job is as slow as the slowest)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_rank: int, world: int, seconds_max: float) -> float:
    """Whole-job GB/s of `world` independent replicas: all bytes over the slowest rank's time."""
    return world * bytes_per_rank / seconds_max / 1e9


def time_events(torch, fn, iters):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    b.synchronize()
    return a.elapsed_time(b)   # ms


# ------------------------------------------------------------------------------------------------
# CPU oracle arm

def oracle_sample_seconds(max_layers=12, M=16, g=128, min_seconds=10.0):
    """Times the oracle, as it stands, on the first layers of the stack (numpy-generated weights):
    layer after layer until at least `min_seconds` of oracle time or `max_layers` layers.
    Returns (seconds, layers)."""
    from oracle import w4a16_oracle as orc
    h = qsynth.stack_h0(M)
    total, n = 0.0, 0
    while n < max_layers and total < min_seconds:
        w = {nm: qsynth.stack_layer_weights(n, nm, g) for nm in qsynth.LAYER_SHAPES}
        t0 = time.perf_counter()
        h, _ = orc.stack_layer_free_running(h, w, g, qsynth.Q_DIM)
        total += time.perf_counter() - t0
        n += 1
    return total, n


def oracle_check_last_layer(step, torch):
    """The configuration that was timed, looked at with the oracle: the five linears of the LAST layer
    of the step just run (its activation buffers still hold that layer's tensors), each recomputed
    from the bf16 input the GPU fed it and from the boundary tensors that the oracle's layout
    reference recovers from the packed weights the kernels streamed.  Part of the CPU-baseline leg."""
    from oracle import w4a16_oracle as orc
    step.run()
    torch.cuda.synchronize()
    u16 = lambda t: t.cpu().numpy().view(np.uint16)
    b, l, g = step.bufs, step.n_layers - 1, step.g
    src = step.h_in if l == 0 else step.h[(l - 1) % 2]
    feeds = {"qkv": (src, b["qkv"]), "o": (b["a"], b["o"]), "gate": (b["r"], b["gt"]), "up": (b["r"], b["up"]), "down": (b["d"], b["dn"])}
    worst_rf, worst_me = 0.0, 0.0
    for nm, (xin, yout) in feeds.items():
        K, N = qsynth.LAYER_SHAPES[nm]
        wq, sc, z = orc.unpack_ref(step.packed[l][nm].cpu().numpy(), K, N, g)
        y64 = orc.qlinear_f64(u16(xin), wq, sc, z, g, col_block=4096)
        y = orc.bf16_bits_to_f64(u16(yout))
        worst_rf = max(worst_rf, float(orc.rel_frobenius(y, y64)))
        worst_me = max(worst_me, float(orc.max_scaled_abs_err(y, y64)))
    ok = worst_rf <= 2e-3 and worst_me <= 1e-2
    assert ok, f"timed configuration fails the oracle: relF {worst_rf:.3e}, max scaled error {worst_me:.3e}"
    return {"layer": l, "linears": 5, "max_rel_frobenius": worst_rf, "max_scaled_abs_err": worst_me, "within_tolerance": ok}


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        n = 1
    return int(min(n, len(os.sched_getaffinity(0))))


def oracle_linear_seconds(w, x_bits, g=128):
    from oracle import w4a16_oracle as orc
    t0 = time.perf_counter()
    orc.f64_to_bf16_bits(orc.qlinear_f64(x_bits, w["wq"], w["scale"], w["zero"], g))
    return time.perf_counter() - t0


def run_reference(args, rank, world):
    """The oracle, as it stands, on the host cores; one step = the fused-qkv linear of layer 0
    (a bounded sample of the verify step, so that any --steps K ends within minutes)."""
    if rank != 0:
        return
    M, g = 16, 128
    K, N = qsynth.LAYER_SHAPES["qkv"]
    w = qsynth.stack_layer_weights(0, "qkv", g)
    x = qsynth.stack_h0(M)
    nbytes = linear_bytes(M, K, N, g)
    for _ in range(args.warmup):
        oracle_linear_seconds(w, x, g)
    t = [oracle_linear_seconds(w, x, g) for _ in range(args.steps)]
    sec = float(np.mean(t))
    val = nbytes / sec / 1e9
    sample = f"fused-qkv linear of layer 0 (M=16, K={K}, N={N}, g=128) per step; {nbytes} algorithmic bytes"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": host_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


METRIC = "W4A16 verify-GEMM HBM GB/s at M=16 (36-layer stack + LM head per step)"
WORKLOAD = ("verify_step: 36-layer W4A16 linear stack (qkv,o,gate,up,down + unit-RMS glue) "
            "+ LM head with arg-max, M=16, g=128, 4B-class shapes")


# ------------------------------------------------------------------------------------------------

def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    import paper_2607_04244_b200 as ql
    ql.load()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    M, g = 16, 128
    step = VerifyStep(ql, torch, M, g, n_layers=args.layers, lm_head=not args.no_lm_head)
    total_bytes, per_layer = step_bytes(M, g, n_layers=args.layers, lm_head=not args.no_lm_head)
    for _ in range(max(args.warmup, 3)):
        step.run()
    torch.cuda.synchronize()
    assert ql.ql_device_status(step.ws) == ql.QL_OK

    # ---- device-resident timing (the headline value) ----
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    t0 = time.time()
    l0 = ql.ql_launch_count()
    h0 = time.perf_counter()
    ms = time_events(torch, step.run, args.steps)
    launches = ql.ql_launch_count() - l0
    t1 = time.time()
    torch.cuda.synchronize()
    # host time to enqueue one step (wall clock of the call alone, GPU idle afterwards)
    h0 = time.perf_counter()
    step.run()
    host_enqueue_ms = (time.perf_counter() - h0) * 1e3
    torch.cuda.synchronize()
    barrier()
    ms_local = ms
    ms = max_over_ranks(ms, world)
    clocks = sampler.stop(t0, t1) if sampler else None
    ms_per_step_local = ms_local / args.steps
    ms_per_step = ms / args.steps
    value = aggregate_value(total_bytes, world, ms_per_step * 1e-3)

    if args.no_extras:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": "GB/s", "ms_per_step": ms_per_step,
                              "layers": args.layers, "host_enqueue_ms": host_enqueue_ms,
                              "gpu_launches": int(launches), "note": "reduced run for profiler captures"}), flush=True)
        return
    # ---- end to end through the host-buffer entry point ----
    for _ in range(2):
        step.run_host()
    barrier()
    w0 = time.perf_counter()
    for _ in range(args.steps):
        step.run_host()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - w0) / args.steps
    e2e_s = max_over_ranks(e2e_s, world)
    e2e_val = aggregate_value(total_bytes, world, e2e_s)

    # ---- dominant kernel: the persistent stack kernel runs the whole step in one launch ----
    # (launch count per step is measured, the kernel time is the CUDA-event time of the timed region)
    peak, peak_kind = measured_peak()
    launches_per_step = max(1, int(round(launches / args.steps)))
    achieved = total_bytes / (ms_per_step_local * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind} (copy bandwidth, burst)", "kernel": "qstack_tc5_kernel",
                "launches_per_step": launches_per_step, "avg_launch_us": ms_per_step_local * 1e3 / launches_per_step,
                "bytes_per_launch": total_bytes / launches_per_step,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": NCU_TRAFFIC_RATIO * total_bytes / launches_per_step,
                "traffic_source": "ncu capture of a 3-layer launch, scaled by algorithmic bytes",
                "note": "one step = a chain of 145 dependent fused operations; each waits for the one before it, "
                        "so the step is bound by dependency latency, not by HBM bandwidth (see single_linear_cold_l2_m16 "
                        "and lm_head_m16 for the same kernel without the chain)"}

    # ---- the step's tokens through both entry points must agree ----
    step.tokens.fill_(-1)
    step.run()
    torch.cuda.synchronize()
    tok_dev = step.tokens.cpu().numpy().copy()
    step.run_host()
    tokens_agree = bool(np.array_equal(tok_dev, step.host_tokens.numpy())) if step.lm is not None else None
    assert tokens_agree is not False, "qlinear_stack_w4a16 and qlinear_stack_w4a16_host returned different tokens"

    # ---- every shape of the step on its own, cold L2: the 36 distinct weight sets of the step, distinct
    #      outputs, back to back (independent operations) ----
    extras, sweep_block, lm_point = {}, [], None
    if step.n_layers >= 24:
        for nm in ("gate", "down", "qkv", "o"):
            K, N = qsynth.LAYER_SHAPES[nm]
            extras[nm] = independent_point(ql, torch, M, K, N, g, [step.packed[l][nm] for l in range(step.n_layers)], step.ws)
        # configuration 4 in brief (the full 84 points: --sweep): M in {1, 16, 64} x the three shapes, g = 128
        ws64 = ql.new_workspace(64, qsynth.MLP_DIM)
        for nm in ("gate", "down", "qkv"):
            K, N = qsynth.LAYER_SHAPES[nm]
            for Ms in (1, 16, 64):
                sweep_block.append(independent_point(ql, torch, Ms, K, N, g, [step.packed[l][nm] for l in range(step.n_layers)],
                                                     ws64 if Ms > 16 else step.ws, iters=3))
        del ws64
    if step.lm is not None:
        # configuration 3: the LM head with its arg-max on its own (207 MB per call: cold by size)
        lm_ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=qsynth.HIDDEN, N=qsynth.VOCAB, g=g, ld_in=qsynth.HIDDEN,
                                   ld_out=qsynth.VOCAB, packed=step.lm, in0=step.h_last, out=None, argmax_out=step.tokens)])
        fn = lambda: ql.qlinear_stack_w4a16(lm_ops, step.ws)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = sorted(time_events(torch, fn, 1) * 1e3 for _ in range(7))
        b = linear_bytes(M, qsynth.HIDDEN, qsynth.VOCAB, g, y_bytes=False) + 4 * M
        lm_point = {"us": ts[len(ts) // 2], "us_min": ts[0], "bytes": b, "GBps": b / ts[len(ts) // 2] / 1e3,
                    "frac_of_measured_peak": b / ts[len(ts) // 2] / 1e3 / peak, "kernel": "qstack_tc5_kernel (tokens only, no Y)"}

    swa_block = swa_points(ql, torch) if (rank == 0 and not args.no_extras) else None

    if rank != 0:
        return
    line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "algorithmic_bytes_per_step": total_bytes, "l2": "inputs (2.15 GB of weights) larger than L2",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "us_per_36_layer_stack_and_lm_head": ms_per_step * 1e3,
            "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "clocks": clocks, "gpu_launches": int(launches), "host_enqueue_ms_per_step": host_enqueue_ms,
            "e2e": {"value": e2e_val, "unit": "GB/s", "h2d_bytes_per_step": int(step.host_in.numel() * 2),
                    "d2h_bytes_per_step": int(step.host_tokens.numel() * 4), "ms_per_step": e2e_s * 1e3},
            "roofline": roofline, "single_linear_cold_l2_m16": extras, "lm_head_m16": lm_point, "m_sweep": sweep_block,
            "drafter_swa_attention": swa_block, "tokens_agree_device_vs_host_entry": tokens_agree}
    if world == 1 and not args.no_cpu_baseline:
        sec, n_sample = oracle_sample_seconds(12, M, g)
        line["cpu_baseline"] = {"value": per_layer * n_sample / sec / 1e9, "unit": "GB/s", "cores": host_threads(),
                                "kind": "oracle", "seconds": sec,
                                "sample": f"layers 0-{n_sample - 1} of the 36-layer stack (M=16, g=128), "
                                          f"{per_layer * n_sample} algorithmic bytes",
                                "timed_run_checked": oracle_check_last_layer(step, torch)}
    print(json.dumps(line), flush=True)


def run_drafter(args):
    """Second workload (paper Sections 3.2, 3.3): the drafter's W4 linears - 5 layers, hidden 2560,
    group-wise symmetric INT4 with groups of 128 (zero == NULL at the boundary), M = 16 - through
    the same launcher.  The projection widths are SYNTHETIC (the target's; the paper does not give
    them).  One step streams 0.27 GB, which fits in L2, so a buffer larger than L2 is written
    between steps.  Prints one JSON line."""
    import torch
    import paper_2607_04244_b200 as ql
    ql.load()
    M, g, L = 16, 128, qsynth.DRAFTER_LAYERS
    step = VerifyStep(ql, torch, M, g, n_layers=L, lm_head=False, symmetric=True)
    per_layer = sum(linear_bytes(M, K, N, g) - (K // g) * N // 2 for (K, N) in qsynth.LAYER_SHAPES.values())   # no zero points
    total = L * per_layer
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    for _ in range(max(args.warmup, 3)):
        step.run()
    torch.cuda.synchronize()
    assert ql.ql_device_status(step.ws) == ql.QL_OK
    ts = []
    for _ in range(args.steps):
        flush.fill_(1)
        ts.append(time_events(torch, step.run, 1))
    ms = float(np.median(ts))
    peak, peak_kind = measured_peak()
    val = total / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "W4A16 drafter-block HBM GB/s at M=16 (5 symmetric-INT4 layers per step)", "value": val,
                      "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "drafter_block: 5 layers x (qkv, o, gate, up, down), symmetric g=128, M=16, "
                                             "synthetic widths (the target's)", "algorithmic_bytes_per_step": total,
                                 "l2": "256 MB written between steps (the step's 0.27 GB would otherwise stay in L2)"},
                      "roofline": {"bound": "hbm", "achieved": val, "peak": peak, "unit": "GB/s", "frac": val / peak,
                                   "peak_kind": f"of {peak_kind}", "kernel": "qstack_tc5_kernel"},
                      "gpu_launches": args.steps + max(args.warmup, 3)}), flush=True)


def run_sweep(args):
    """M-sweep: M x three shapes x g in {64,128} x zero mode; one JSON line per point."""
    import torch
    import paper_2607_04244_b200 as ql
    ql.load()
    reps = 36     # distinct weight buffers per point (as in the default bench line): 36 x >= 8 MB > 2 x L2
    for si, (K, N) in enumerate(qsynth.SWEEP_SHAPES):
        for g in (128, 64):
            for sym in (False, True):
                packed = [device_linear(ql, torch, 7000 + 100 * si + r, K, N, g, sym) for r in range(reps)]
                ws = ql.new_workspace(64, N)
                for M in qsynth.SWEEP_M:
                    row = independent_point(ql, torch, M, K, N, g, packed, ws, sym=sym, iters=7)
                    row["sweep"] = True
                    print(json.dumps(row), flush=True)
                del packed, ws
                torch.cuda.empty_cache()


def run_paths(args):
    """Path comparison behind ql_select_path: the warp-level mma.sync kernel and the tcgen05 kernel,
    one launch per linear (forced path), 24 distinct weight sets back to back; one JSON line per point."""
    import torch
    import paper_2607_04244_b200 as ql
    ql.load()
    g, reps = 128, 24
    for (K, N) in qsynth.SWEEP_SHAPES:
        packed = [device_linear(ql, torch, 9000 + r, K, N, g) for r in range(reps)]
        ws = ql.new_workspace(64, N)
        for M in qsynth.SWEEP_M:
            xin = torch.randn((M, K), device="cuda").to(torch.bfloat16).view(torch.int16)
            yout = torch.zeros((M, N), dtype=torch.int16, device="cuda")
            row = {"paths": True, "M": M, "K": K, "N": N, "g": g}
            for path, name in ((ql.QL_PATH_MMA, "mma"), (ql.QL_PATH_TC5, "tcgen05")):
                def fn():
                    for p in packed:
                        ql.qlinear_w4a16(p, xin, yout, None, M, K, N, g, ws, path=path)
                try:
                    for _ in range(2):
                        fn()
                    torch.cuda.synchronize()
                    ts = sorted(time_events(torch, fn, 1) / reps * 1e3 for _ in range(7))
                    row[f"us_{name}"] = ts[len(ts) // 2]
                except ql.QlError as e:
                    row[f"us_{name}"] = None
                    row[f"{name}_status"] = e.status
            row["selected"] = ql.PATH_NAMES[ql.ql_select_path(M, K, N, g)]
            print(json.dumps(row), flush=True)
        del packed
        torch.cuda.empty_cache()


def run_linears(args):
    """R independent linears of one shape (distinct weights and outputs) in one stack call: the
    launcher sends them to the batch kernel.  Prints one JSON line."""
    import torch
    import paper_2607_04244_b200 as ql
    ql.load()
    K, N, R = (int(v) for v in args.linears.split(","))
    M, g = 16, 128
    packed = [device_linear(ql, torch, 8000 + r, K, N, g) for r in range(R)]
    ws = ql.new_workspace(M, N)
    xin = torch.randn((M, K), device="cuda").to(torch.bfloat16).view(torch.int16)
    youts = [torch.zeros((M, N), dtype=torch.int16, device="cuda") for _ in range(R)]
    ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=p, in0=xin, out=y)
                       for p, y in zip(packed, youts)])
    plan = ql.ql_stack_plan(ops, ws.data_ptr(), ws.numel())
    if args.path == "stack":
        fn = lambda: ql.qlinear_stack_w4a16(ops, ws)
    else:
        forced = ql.QL_PATH_MMA if args.path == "mma" else ql.QL_PATH_TC5

        def fn():
            for pk, y in zip(packed, youts):
                ql.qlinear_w4a16(pk, xin, y, None, M, K, N, g, ws, path=forced)
        plan = {"one launch per linear": args.path}
    for _ in range(max(args.warmup, 3)):
        fn()
    torch.cuda.synchronize()
    us = time_events(torch, fn, args.steps) / args.steps / R * 1e3
    b = linear_bytes(M, K, N, g)
    print(json.dumps({"workload": f"{R} independent linears 16x{K}x{N} g128, distinct weights (cold L2)", "us_per_linear": us,
                      "GBps": b / us / 1e3, "frac_of_8TBs": b / us / 1e3 / NOMINAL_HBM_GBS, "plan": plan,
                      "status": ql.ql_device_status(ws)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--swa", action="store_true", help="only the drafter's sliding-window attention points, one JSON line")
    ap.add_argument("--workload", default="verify_step", choices=["verify_step", "drafter"],
                    help="drafter: the second workload (5 symmetric-INT4 layers, synthetic widths)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=qsynth.N_LAYERS,
                    help="layers of the stack (default: the full 36; smaller values are for profiler captures)")
    ap.add_argument("--no-lm-head", action="store_true", help="leave the LM head out (profiler captures)")
    ap.add_argument("--no-extras", action="store_true", help="skip the single-linear and end-to-end legs")
    ap.add_argument("--paths", action="store_true", help="forced-path comparison (mma.sync vs tcgen05), one launch per linear")
    ap.add_argument("--path", default="stack", choices=["stack", "mma", "tcgen05"],
                    help="with --linears: one stack call (default) or one forced-path qlinear_w4a16 launch per linear")
    ap.add_argument("--linears", default=None, metavar="K,N,R",
                    help="instead of the verify step: R independent 16xKxN linears in one call (batch kernel)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.workload == "drafter":
        run_drafter(args)
        return
    if args.swa:
        import torch
        import paper_2607_04244_b200 as ql
        ql.load()
        print(json.dumps({"drafter_swa_attention": swa_points(ql, torch), "gpu_launches": int(ql.ql_launch_count())}), flush=True)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.paths:
        run_paths(args)
        return
    if args.linears:
        run_linears(args)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
