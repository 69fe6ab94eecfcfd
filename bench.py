#!/usr/bin/env python
"""Benchmark of the block-sparse video attention hot path on B200.

One step = one pass of the whole path over one batch of synthetic Q/K/V: block routing
(pool -> scores -> select -> CSR) followed by block-sparse attention over the kept blocks.
`value` is effective TFLOP/s on the selected blocks (4*Bs^2*d FLOP per kept tile) with the
inputs resident in HBM; `e2e` is the same metric with the step's Q/K/V copied from pinned host
memory and O copied back inside the timed region.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large] [--impl reference]

With N > 1 (torchrun) every rank is a replica working on its own batch sample: no data-path
collective, weak scaling, time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2606_23743_b200 import dist as D  # noqa: E402
from paper_2606_23743_b200.workloads import SEED_BASE, WORKLOADS, bf16_bits, make_prologue_inputs, make_qkv  # noqa: E402

METRIC = "block-sparse attn fwd effective TFLOPS (selected blocks)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, constants copied from one ncu capture each
# (`ncu --set full --clock-control none -k regex:<kernel> -c 1` of this script on the "large" workload);
# they are not measured by this run.  Other workloads: not captured (null).
ATTN_TRAFFIC_BYTES = {"large": 793.9e6}           # attn_ts_kernel, V read where it lies (605.4 MB read + 188.5 MB written)
TRANSPOSE_TRAFFIC_BYTES = {"large": 355.9e6}      # transpose_v_kernel (201.3 MB read + 154.6 MB written)
SM_COUNT_FALLBACK = 148


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.max_mhz, self.power = [], set(), None, []
        self.period_s = period_s
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(device_index)
            handle = None
            uuid = getattr(props, "uuid", None)
            if uuid is not None:
                try:
                    handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    handle = None
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv, self._h = pynvml, handle
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report no samples rather than fail the bench
            self._nv, self._h, self.error = None, None, repr(e)

    def _names(self, mask):
        nv = self._nv
        table = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
                 "hw_power_brake": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80)}
        return {k for k, bit in table.items() if mask & bit}

    def _run(self):
        nv, h = self._nv, self._h
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                self.reasons |= self._names(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period_s)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        # NVML's clock and power readings lag by tens of milliseconds: a record of fewer than ~100 samples
        # (a burst of a few dozen ms) describes the idle GPU before the burst, not the burst
        return {"sm_mhz": med, "sm_mhz_min": float(min(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "power_w_max": max(self.power) if self.power else None,
                "reliable": len(self.samples) >= 100}


def flops_per_tile(w):
    return 4.0 * w.block * w.block * w.d


# ------------------------------------------------------------------ CPU oracle legs
def oracle_sample(w, qb, kb, vb, n_rows):
    """Times the oracle, as it stands, on the first n_rows query-block rows of batch 0 (whole
    heads first): pooling, scores and selection of the heads touched, then attention of those
    rows.  Returns (seconds, flops, rows)."""
    import oracle
    n_rows = max(1, min(n_rows, w.H * w.Nb))
    heads = -(-n_rows // w.Nb)
    q1, k1, v1 = qb[:1, :heads], kb[:1, :heads], vb[:1, :heads]
    t0 = time.perf_counter()
    if w.fp8:       # FP8 variant: the quantiser is part of the path; routing and attention see the dequantised values
        q1 = oracle.dequantize_e4m3(*oracle.quantize_e4m3(q1, w.N, w.block), w.N, w.block)
        k1 = oracle.dequantize_e4m3(*oracle.quantize_e4m3(k1, w.N, w.block), w.N, w.block)
    sel, _ = oracle.select_from_qk(q1, k1, w.N, w.block, w.scale, w.mode, w.k, w.tau, w.win_t, w.win_s,
                                   w.blocks_per_frame if w.win_t >= 0 else 0)
    rows = list(range(n_rows))
    oracle.attn_rows(q1, k1, v1, w.N, w.block, w.scale, sel.row_ptr, sel.col_idx, rows=rows)
    dt = time.perf_counter() - t0
    nnz = int(sel.row_ptr[n_rows] - sel.row_ptr[0])
    return dt, nnz * flops_per_tile(w), n_rows


def cpu_baseline(w, qb, kb, vb, target_s=15.0):
    import oracle
    dt, fl, n = oracle_sample(w, qb, kb, vb, 32)
    per_row = max(dt / max(n, 1), 1e-6)
    n_rows = int(min(w.H * w.Nb, max(32, target_s / per_row)))
    dt, fl, n = oracle_sample(w, qb, kb, vb, n_rows)
    return {"value": fl / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"'{w.name}', batch 0: routing of the first {-(-n // w.Nb)} head(s) and attention of "
                      f"their first {n} query-block rows; {dt:.1f} s wall",
            "seconds": dt}


def run_reference(args):
    rank, _, world = D.env_world()
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = WORKLOADS[args.workload]
    from paper_2606_23743_b200.workloads import shrink
    w1 = shrink(w, B=1, H=min(w.H, 4))
    q, k, v = make_qkv(w1, SEED_BASE + w.cfg)
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    total = args.steps + args.warmup
    dt, fl, n = oracle_sample(w1, qb, kb, vb, 16)
    per_row = max(dt / n, 1e-6)
    n_rows = int(min(w1.H * w1.Nb, max(4, (150.0 / max(total, 1)) / per_row)))
    for _ in range(args.warmup):
        oracle_sample(w1, qb, kb, vb, n_rows)
    t0 = time.perf_counter()
    flops = 0.0
    for _ in range(args.steps):
        _, fl, n = oracle_sample(w1, qb, kb, vb, n_rows)
        flops += fl
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "d": w.d, "N": w.N, "block": w.block,
                   "rule": "mass>=%.2f cap %d" % (w.tau, w.k) if w.mode == 1 else "top-%d" % w.k,
                   "parallelism": "host cores", "prologue": False,
                   "note": "fp64 CPU oracle on host cores; each step is a bounded sample of this workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"per step: routing of the first {-(-n // w.Nb)} head(s) + attention of their first {n} query-block rows"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ GPU arm
def two_step_wanted(args, w):
    """--v-copy: the two-step form of plain bf16 attention (the other forms have no such step)."""
    return bool(args.v_copy) and not w.fp8 and not args.fp4 and not args.remainder


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=list(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--fp4", action="store_true",
                    help="extended step: Q and K quantised to 4-bit block-scaled codes inside every step, Q K^T as a "
                         "block-scaled 4-bit MMA (routing stays on the bf16 Q, K); 128-token blocks only")
    ap.add_argument("--remainder", action="store_true",
                    help="extended step: attention with the approximate remainder of the dropped blocks (order 0) "
                         "instead of exact-only attention; `value` still counts the selected blocks' FLOPs only")
    ap.add_argument("--remainder-order", type=int, default=0, choices=[0, 1],
                    help="with --remainder: 0 = block-mean term only, 1 = plus the first-order term")
    ap.add_argument("--sustained-seconds", type=float, default=2.5,
                    help="length of the second, back-to-back leg whose clocks NVML can follow (0 = skip)")
    ap.add_argument("--v-copy", action="store_true",
                    help="bf16: the two-step form -- a tiled transposed copy of V made on a second stream beside routing, "
                         "then the attention kernel on that copy (default: one call that reads V where it lies)")
    ap.add_argument("--prologue", action="store_true",
                    help="extended step: the fused QK-norm + RoPE prologue in front (it also writes the block means, "
                         "and the e4m3 codes of an FP8 workload, so routing skips its pooling pass and the quantiser)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    from paper_2606_23743_b200 import binding as B
    from paper_2606_23743_b200 import build as build_mod
    build_mod.build()
    B.lib()                                       # fail loudly if the CUDA library is missing

    rank, local_rank, world = D.init()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    w = WORKLOADS[args.workload]
    warmup = max(args.warmup, 3)

    qh, kh, vh = (x.pin_memory() for x in make_qkv(w, D.rank_seed(SEED_BASE + w.cfg, rank)))
    q, k, v = (x.to(dev, non_blocking=True) for x in (qh, kh, vh))
    o = torch.empty_like(v)
    oh = torch.empty(o.shape, dtype=o.dtype).pin_memory()
    p = B.make_problem(q, k, v, o, w.N, w.block)
    pq = B.make_problem(q, k, None, None, w.N, w.block)
    if args.prologue:
        gq, gk, cos_t, sin_t = (x.to(dev) for x in make_prologue_inputs(w))
        qn, kn = torch.empty_like(q), torch.empty_like(k)
        qm = torch.empty(w.B, w.H, w.Nb, w.d, dtype=torch.float32, device=dev)
        km = torch.empty_like(qm)
    if w.fp8:
        # FP8 variant: Q and K are quantised to e4m3 with per-block scales inside every step
        q8, k8 = torch.zeros(q.shape, dtype=torch.uint8, device=dev), torch.zeros(k.shape, dtype=torch.uint8, device=dev)
        qs = torch.zeros(w.B, w.H, w.Nb, dtype=torch.float32, device=dev)
        ks = torch.zeros_like(qs)
        p = B.make_problem(q8, k8, v, o, w.N, w.block, 0.0, True)
    s = B.make_select(w.mode, w.k, w.tau, w.win_t, w.win_s, w.blocks_per_frame if w.win_t >= 0 else 0)
    ws = torch.empty(max(B.select_workspace_bytes(p, s), 256), dtype=torch.uint8, device=dev)
    row_ptr = torch.zeros(w.R + 1, dtype=torch.int32, device=dev)
    col_idx = torch.zeros(B.select_max_nnz(p, s), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if args.remainder and (w.fp8 or args.prologue):
        raise SystemExit("--remainder runs on the plain bf16 step")
    if args.fp4:
        if w.fp8 or args.prologue or args.remainder or w.block != 128 or w.d != 128:
            raise SystemExit("--fp4 runs on a bf16 workload with 128-token blocks and d = 128")
        BH = w.B * w.H
        q4 = torch.zeros(BH, w.Nb * 128, 64, dtype=torch.uint8, device=dev); k4 = torch.zeros_like(q4)
        qsf = torch.zeros(BH, w.Nb, 1024, dtype=torch.uint8, device=dev); ksf = torch.zeros_like(qsf)
        qg = torch.zeros(BH, dtype=torch.float32, device=dev); kg = torch.zeros_like(qg)
        ws4 = torch.zeros(max(8 * BH, 256), dtype=torch.uint8, device=dev)
    # the one-call entry points read V where it lies and need only their row counters (and tile lists);
    # the two-step form (--v-copy) keeps a transposed copy of V in the workspace
    aws_bytes = (B.attn_remainder_workspace_bytes(p, args.remainder_order) if args.remainder else 256 if args.fp4 else
                 B.attn_workspace_bytes(p) if args.v_copy else B.attn_one_call_workspace_bytes(p))
    aws = torch.empty(max(aws_bytes, 256), dtype=torch.uint8, device=dev)
    # the first-order term of the remainder weighs the dropped blocks by the routing's scores
    scores_buf = (torch.empty(w.B, w.H, w.Nb, w.Nb, dtype=torch.float32, device=dev)
                  if args.remainder and args.remainder_order == 1 else None)
    variable_rows = w.mode == 1 or (w.win_t >= 0 and w.k < (2 * w.win_t + 1) * (2 * w.win_s + 1))
    # routing kernels (pooling, scores, selection; CSR assembly when rows vary in length) + V transpose
    # + attention (+ the tile-list kernel of the 64-token-block path, + the quantiser of the FP8 variant)
    launches_per_step = (4 if variable_rows else 3) + 2 + (1 if w.block == 64 else 0) + (1 if w.fp8 else 0)
    if not two_step_wanted(args, w):   # no V transpose: V is read where it lies
        launches_per_step -= 1
    if args.prologue:       # + the prologue, - the pooling kernel, - the quantiser
        launches_per_step += 1 - 1 - (1 if w.fp8 else 0)
    if args.fp4:            # + amax and cast kernels of the 4-bit quantiser
        launches_per_step += 2
    if args.remainder:      # + the block means of K and V (the memset before it is not a kernel of this library)
        launches_per_step += 1 + (3 if args.remainder_order == 1 else 0)       # order 1: + C_J, weights, aggregation

    # V is prepared (tiled transposed copy) on a second stream while routing, which never reads V, runs
    # (lower priority: its CTAs fill the SMs that the latency-bound selection kernel leaves idle instead of
    # competing with the HBM-bound pooling kernel)
    main = torch.cuda.Stream(priority=-1)
    side = torch.cuda.Stream(priority=0)
    main.wait_stream(torch.cuda.current_stream())
    torch.cuda.set_stream(main)
    v_ready = torch.cuda.Event()

    def prepare_v(vv):
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            B.attn_prepare_v(p, vv, aws)
            v_ready.record()

    # the two-step form serves what the tensor-core kernel serves (every supported shape today)
    # bf16: V is prepared (tiled transposed copy) beside routing; the other forms have no such step
    two_step = args.v_copy and B.attn_workspace_bytes(p) > 0 and not args.remainder and not args.fp4 and not w.fp8

    def route(qq, kk, vv):
        if args.prologue:
            if two_step:
                prepare_v(vv)
            if w.fp8:
                B.qk_norm_rope_pool(pq, qq, kk, gq, gk, cos_t, sin_t, 1e-6, qn, kn, qm, km, q8, k8, qs, ks)
            else:
                B.qk_norm_rope_pool(pq, qq, kk, gq, gk, cos_t, sin_t, 1e-6, qn, kn, qm, km)
            B.block_select_pooled(p, s, qm, km, row_ptr, col_idx, ws)
        elif w.fp8:
            if two_step:
                prepare_v(vv)
            B.quantize_qk_fp8(pq, qq, kk, q8, k8, qs, ks)
            B.block_select(p, s, q8, k8, row_ptr, col_idx, ws, qs, ks)
        else:
            if two_step:
                prepare_v(vv)
            B.block_select(p, s, qq, kk, row_ptr, col_idx, ws, block_scores=scores_buf)

    def attend(qq, kk, vv, oo):
        if args.prologue:
            qq, kk = qn, kn
        if args.fp4:
            B.quantize_qk_fp4(pq, qq, kk, q4, k4, qsf, ksf, qg, kg, ws4)
            B.block_sparse_attn_fwd_fp4(p, q4, k4, qsf, ksf, qg, kg, vv, row_ptr, col_idx, oo, None, status, aws)
        elif args.remainder:
            B.block_sparse_attn_remainder_fwd(p, qq, kk, vv, row_ptr, col_idx, oo, None, status, args.remainder_order, aws,
                                              scores_buf)
        elif w.fp8 and two_step:
            torch.cuda.current_stream().wait_event(v_ready)
            B.block_sparse_attn_fwd_prepared(p, q8, k8, row_ptr, col_idx, oo, None, status, workspace=aws,
                                             q_scale=qs, k_scale=ks)
        elif w.fp8:
            B.block_sparse_attn_fwd(p, q8, k8, vv, row_ptr, col_idx, oo, None, status, qs, ks, workspace=aws)
        elif two_step:
            torch.cuda.current_stream().wait_event(v_ready)
            B.block_sparse_attn_fwd_prepared(p, qq, kk, row_ptr, col_idx, oo, None, status, workspace=aws)
        else:
            B.block_sparse_attn_fwd(p, qq, kk, vv, row_ptr, col_idx, oo, None, status, workspace=aws)

    def step():
        route(q, k, v)
        attend(q, k, v, o)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    nnz = int(row_ptr[-1].item())
    assert int(status.item()) == 0, "device status set during warm-up"
    step_flops = nnz * flops_per_tile(w)

    # ---- device-resident timing
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sel_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    att_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    D.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for i in range(args.steps):
        sel_ev[i][0].record()
        route(q, k, v)
        sel_ev[i][1].record()
        att_ev[i][0].record()
        attend(q, k, v, o)
        att_ev[i][1].record()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    D.barrier()
    total_ms = D.max_over_ranks(ev0.elapsed_time(ev1))
    ms_per_step = total_ms / args.steps
    attn_ms = float(np.mean([a.elapsed_time(b) for a, b in att_ev]))
    sel_ms = float(np.mean([a.elapsed_time(b) for a, b in sel_ev]))
    job_flops = D.sum_over_ranks(step_flops)
    value = job_flops / (ms_per_step * 1e-3) / 1e12
    assert int(status.item()) == 0, "device status set during the timed region"

    # ---- the same step back to back for seconds: the regime a denoising loop lives in (the part is
    # power-limited, so the SM clock settles below its burst value) and the only one NVML's readings can
    # follow.  Same work per step as above; nothing of it enters `value`.
    sms = torch.cuda.get_device_properties(local_rank).multi_processor_count or SM_COUNT_FALLBACK
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = max(args.steps, int(args.sustained_seconds * 1e3 / ms_per_step) + 1)
        s_att = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_sus)]
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sus_sampler = ClockSampler(local_rank, period_s=0.005)
        D.barrier()
        torch.cuda.synchronize()
        s0.record()
        for i in range(n_sus):
            route(q, k, v)
            s_att[i][0].record()
            attend(q, k, v, o)
            s_att[i][1].record()
            if i == n_sus // 5:
                sus_sampler.start()               # sample the settled part only (the first fifth ramps down)
        s1.record()
        torch.cuda.synchronize()
        sus_clocks = sus_sampler.stop()
        D.barrier()
        sus_ms = D.max_over_ranks(s0.elapsed_time(s1)) / n_sus
        tail = s_att[n_sus // 5:]
        sus_attn_ms = float(np.mean([a.elapsed_time(b) for a, b in tail]))
        mhz = sus_clocks["sm_mhz"]
        sustained = {"seconds": sus_ms * n_sus * 1e-3, "steps": n_sus, "ms_per_step": sus_ms,
                     "value": job_flops / (sus_ms * 1e-3) / 1e12, "attention_ms": sus_attn_ms,
                     "attention_tflops": step_flops / (sus_attn_ms * 1e-3) / 1e12,
                     "sm_mhz_median": mhz, "sm_mhz_min": sus_clocks["sm_mhz_min"],
                     "power_w_max": sus_clocks["power_w_max"], "reasons": sus_clocks["reasons"],
                     "clock_samples": sus_clocks["samples"],
                     "cycles_per_tile": sus_attn_ms * 1e-3 * mhz * 1e6 * sms / nnz if mhz else None,
                     "note": "attention_ms, clocks and power over the last four fifths of the leg"}
        assert int(status.item()) == 0, "device status set during the sustained leg"

    # ---- the kernel's own cycle counter (one extra launch): cycles do not depend on the SM clock, so
    # cycles / measured time is the clock each regime really ran at -- the record NVML cannot give for a burst
    kernel_cycles = None
    if B.attn_workspace_bytes(p) > 0:
        prof = torch.zeros(320, dtype=torch.int64, device=dev)
        B.debug_set_prof_buffer(prof)
        try:
            route(q, k, v)
            attend(q, k, v, o)
            torch.cuda.synchronize()
        finally:
            B.debug_set_prof_buffer(None)
        kernel_cycles = int(prof[319].item())

    # ---- attention with its V preparation in line (the one-call entry point: transpose, then the kernel)
    inline_ms = None
    if two_step and not w.fp8 and not args.prologue:
        n_in = max(5, min(args.steps, 20))
        route(q, k, v)
        torch.cuda.current_stream().wait_event(v_ready)
        i0, i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(n_in + 3):
            if i == 3:
                i0.record()
            B.block_sparse_attn_fwd(p, q, k, v, row_ptr, col_idx, o, None, status, workspace=aws)
        i1.record()
        torch.cuda.synchronize()
        inline_ms = i0.elapsed_time(i1) / n_in

    # ---- end to end: pinned host -> device, path, device -> pinned host, every step
    e2e = None
    if not args.no_e2e:
        h2d = sum(x.numel() * x.element_size() for x in (qh, kh, vh))
        d2h = oh.numel() * oh.element_size()
        e_steps = max(3, min(args.steps, 10))

        # Every step copies its Q, K, V from pinned host memory and its O back.  Two sets of device buffers
        # and one copy stream per direction let step i+1's inputs arrive, and step i-1's output leave, while
        # step i computes (PCIe is full duplex); a step still starts only when its own inputs are complete.
        sets = [(q, k, v, o), tuple(torch.empty_like(x) for x in (q, k, v, o))]
        cur = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        in_done = [torch.cuda.Event() for _ in sets]
        comp_done = [torch.cuda.Event() for _ in sets]
        out_done = [torch.cuda.Event() for _ in sets]

        def e2e_steps(n):
            for i in range(n):
                b = i % 2
                qq, kk, vv, oo = sets[b]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(comp_done[b])          # the step that last used these inputs has finished
                    qq.copy_(qh, non_blocking=True); kk.copy_(kh, non_blocking=True); vv.copy_(vh, non_blocking=True)
                    in_done[b].record()
                cur.wait_event(in_done[b])
                if i >= 2:
                    cur.wait_event(out_done[b])                # its previous output has left the device
                route(qq, kk, vv)
                attend(qq, kk, vv, oo)
                comp_done[b].record()
                with torch.cuda.stream(s_out):
                    s_out.wait_event(comp_done[b])
                    oh.copy_(oo, non_blocking=True)
                    out_done[b].record()
            cur.wait_stream(s_out)
            cur.wait_stream(s_in)

        e2e_steps(2)
        torch.cuda.synchronize()
        D.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        e2e_steps(e_steps)
        e1.record()
        torch.cuda.synchronize()
        D.barrier()
        e_ms = D.max_over_ranks(e0.elapsed_time(e1)) / e_steps
        # same inputs every step: what came back must be what the device-resident steps left in o
        assert torch.equal(oh, o.cpu()), "end-to-end output differs from the device-resident result"
        e2e = {"value": job_flops / (e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": e_steps}

    peaks, peak_kind = load_peaks()
    peak = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    achieved = step_flops / (attn_ms * 1e-3) / 1e12
    sel_bytes = 4.0 * w.B * w.H * w.N * w.d
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "e4m3 QK^T, bf16 PV" if w.fp8 else ("e2m1 block-scaled QK^T, bf16 PV" if args.fp4 else "bf16"),
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "d": w.d, "N": w.N, "block": w.block,
                   "rule": "mass>=%.2f cap %d" % (w.tau, w.k) if w.mode == 1 else "top-%d" % w.k,
                   "nnz_tiles": nnz, "parallelism": f"replicas x{world}", "prologue": bool(args.prologue),
                   "remainder": ("order %d: +%d pooled%s tiles per query-block row" % (
                       args.remainder_order, -(-w.Nb // 128), " +%d first-order" % (2 if w.block == 64 else 1)
                       if args.remainder_order else "")) if args.remainder else None,
                   "l2": "inputs (%.0f MB) larger than L2; no flush" % (3 * sel_bytes / 2 / 1e6)},
        "tokens_per_s": world * w.B * w.N / (ms_per_step * 1e-3),
        "attention_ms": attn_ms, "select_ms": sel_ms,
        "attention_tflops": achieved,
        "select_gbs": sel_bytes / (sel_ms * 1e-3) / 1e9,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": ATTN_TRAFFIC_BYTES.get(w.name),
                     "traffic_source": "constant from one ncu capture of attn_ts_kernel on this workload, not measured by this run",
                     "traffic_with_v_transpose": (ATTN_TRAFFIC_BYTES[w.name] + TRANSPOSE_TRAFFIC_BYTES[w.name])
                     if two_step and w.name in ATTN_TRAFFIC_BYTES and w.name in TRANSPOSE_TRAFFIC_BYTES else None,
                     "algorithmic_bytes": 8.0 * w.B * w.H * w.N * w.d,
                     "frac_with_prepare": (step_flops / (inline_ms * 1e-3) / 1e12 / peak) if inline_ms else None,
                     "attention_with_prepare_ms": inline_ms,
                     "frac_whole_step": value / world / peak,
                     "kernel_cycles": kernel_cycles,
                     "cycles_per_tile": kernel_cycles * min(sms, w.R) / nnz if kernel_cycles else None,
                     "cycles_source": "clock64 of the longest CTA of one extra launch (sva_debug_set_prof_buffer)",
                     "sm_mhz_implied_burst": kernel_cycles / (attn_ms * 1e3) if kernel_cycles else None,
                     "sm_mhz_implied_sustained": kernel_cycles / (sustained["attention_ms"] * 1e3)
                     if kernel_cycles and sustained else None,
                     "kernel": "attn_ts_kernel" + (" (the V transpose runs beside routing on a second stream)" if two_step
                                                  else ", V read where it lies"),
                     "mixed_precision_ceiling": peak * 4.0 / 3.0 if w.fp8 else None,
                     "peak_source": f"{peak_kind} bf16 burst",
                     "frac_of_sustained": achieved / float(peaks["bf16_tflops_sustained"])
                     if "bf16_tflops_sustained" in peaks else None,
                     "frac_of_nominal_2250": achieved / 2250.0},
        "clocks": clocks, "sustained": sustained, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline and not args.prologue and not args.remainder and not args.fp4:   # (the oracle leg times the plain step)
            import oracle
            oracle.build()
            line["cpu_baseline"] = cpu_baseline(w, bf16_bits(qh), bf16_bits(kh), bf16_bits(vh))
        print(json.dumps(line))
    D.finalize()


if __name__ == "__main__":
    main()
