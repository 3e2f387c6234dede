#!/usr/bin/env python
"""Benchmark of the 2:4 sparse hot path on B200: prune -> compress -> sparse tensor-core GEMM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of seeded synthetic input of the
GPT-3-scale FFN configuration (A 49152 x 12288 bf16, 8192 tokens, beta = 1): pruning and
compression (sp24_prune_compress: the outputs of sp24_prune and sp24_compress from one pass over A,
metadata in the tensor-core layout) and sp24_gemm.  `value` is the dense-equivalent
throughput 2*M*N*K / step time, inputs resident in HBM.  `e2e` is the same metric through the
host-buffer entry point (host -> device copies of A, B, C and the copy of D back inside the
timed region).  `roofline` describes the dominant kernel (the sparse GEMM), timed with CUDA
events inside the timed steps.  `cpu_baseline` times the CPU oracle on a bounded sample of the
same workload.  With --gpus N > 1 (under torchrun) every rank runs the same weight against its
own 8192 tokens (weak scaling, no data-path collective); the time is the max over ranks.

`--impl reference` times the CPU oracle alone on the host cores (a deliberately plain program:
the ratio against it says nothing about kernel quality).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2104_08378_b200 import inputs  # noqa: E402

METRIC = "2:4 sparse GEMM dense-equivalent TFLOPS (prune + compress in one pass, then sp24_gemm, per step)"
UNIT = "TFLOP/s"
NOMINAL_SPARSE_BF16_TFLOPS = 4500.0   # 2 x the 2.25 PFLOP/s dense bf16 datasheet figure
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def ncu_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu summary (profiles/roofline_traffic.json)."""
    path = os.path.join(ROOT, "profiles", "roofline_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        table = json.load(f)
    return table.get(kernel, {}).get(workload)


# -------------------------------------------------------------------------------------------
# clocks during the timed region
# -------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [v for v in visible.split(",") if v.strip() != ""]
                if index < len(ids) and ids[index].isdigit():
                    phys = int(ids[index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nvml = None

    def _run(self):
        n = self.nvml
        while not self._stop.is_set():
            try:
                self.samples.append(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                self.reason_bits |= int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nvml is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples)}


# -------------------------------------------------------------------------------------------
# CPU oracle legs
# -------------------------------------------------------------------------------------------
def oracle_sample(cfg, budget_s: float = 15.0, tile: int = 128):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: compress of the
    A rows the sampled output tiles need, then the sparse GEMM of those tiles.  Returns
    (dense-equivalent TFLOP/s, description, threads)."""
    import oracle
    tiles = inputs.sample_tiles(cfg, 1024, tile)
    # calibrate on one tile, then take as many tiles as fit the budget
    done, t_total, flop = 0, 0.0, 0.0
    target = 1
    while done < len(tiles):
        batch = tiles[done:done + target]
        for (tm, tn) in batch:
            A = inputs.gen_A(cfg, rows=(tm * tile, (tm + 1) * tile))
            Bt = inputs.gen_Bt(cfg, cols=(tn * tile, (tn + 1) * tile))
            t1 = time.perf_counter()
            vals, meta, _ = oracle.compress(A, cfg.ab_type)
            Cm = None
            if cfg.beta != 0:
                Cm = np.ascontiguousarray(inputs.gen_C(cfg, rows=(tm * tile, (tm + 1) * tile))[:, tn * tile:(tn + 1) * tile])
            oracle.gemm_sparse(vals, meta, Bt, cfg.ab_type, cfg.alpha, cfg.beta, Cm,
                               cfg.cd_type if Cm is not None else None)
            t_total += time.perf_counter() - t1          # generation of inputs is not timed
            flop += 2.0 * tile * tile * cfg.K
        done += len(batch)
        per_tile = t_total / done
        remaining = budget_s - t_total
        if remaining <= per_tile:
            break
        target = max(1, min(len(tiles) - done, int(remaining / per_tile)))
    desc = (f"{done} seeded {tile}x{tile} output tiles of {cfg.name} (K={cfg.K}): oracle compress of their "
            f"A rows + oracle sparse GEMM, {t_total:.1f} s")
    return flop / t_total / 1e12, desc, oracle.num_threads()


def run_reference(args, cfg):
    """The reference arm: the CPU oracle on bounded samples of the workload, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    per_step_budget = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(cfg, per_step_budget)
    vals, t0 = [], time.perf_counter()
    desc, threads = "", 1
    for _ in range(args.steps):
        v, desc, threads = oracle_sample(cfg, per_step_budget)
        vals.append(v)
    elapsed = time.perf_counter() - t0
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * elapsed / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": cfg.name, "M": cfg.M, "N": cfg.N, "K": cfg.K,
                                        "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# -------------------------------------------------------------------------------------------
# GPU arm
# -------------------------------------------------------------------------------------------
def run_ours(args, cfg):
    import torch
    from paper_2104_08378_b200 import build
    build.build_library()          # no-op when libsp24.so is newer than its sources; there is no fallback
    from paper_2104_08378_b200 import binding as sp
    from paper_2104_08378_b200 import distributed as D

    rank, local_rank, world = D.init("nccl")
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ab, cd = cfg.ab_type, cfg.cd_type
    tdt = sp.TORCH_DTYPE

    def dev_tensor(a, dt):
        if dt in ("f16", "bf16"):
            return torch.from_numpy(a.view(np.int16)).to(dev).view(tdt[dt])
        return torch.from_numpy(a).to(dev)

    # ---- seeded synthetic inputs (host generator), rank r owns tokens [r*N, (r+1)*N) ----
    M, N, K = cfg.M, cfg.N, cfg.K
    A_h = inputs.gen_A(cfg)
    Bt_h = inputs.gen_Bt(cfg, cols=(rank * N, (rank + 1) * N))
    C_h = None
    if cfg.beta != 0:
        C_h = inputs._matrix(cfg.c_dist, cd, cfg.seed + 7919 * rank, inputs.TENSOR_C, N, 0, M)
    A = dev_tensor(A_h, ab)
    Bt = dev_tensor(Bt_h, ab)
    C = dev_tensor(C_h, cd) if C_h is not None else None
    A_pruned = torch.empty_like(A)
    vals = torch.empty((M, K // 2), dtype=A.dtype, device=dev)
    meta = torch.empty(sp.meta_bytes(ab, M, K, sp.META_TCGEN05), dtype=torch.uint8, device=dev)
    Dout = torch.empty((M, N), dtype=tdt[cd], device=dev)
    ws = torch.zeros(256, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    gemm_events = []

    def check_status(where):
        # the status record is sticky: one read covers every launch since the last read
        if sp.gemm_status(ws) != 0:
            raise SystemExit(f"sp24_gemm reported a device-side timeout ({where})")

    def step(record=False):
        # Section 4.1 step 2 and Section 3.1 in one pass over A: pruned matrix, kept values, metadata
        sp.prune_compress(A, layout=sp.META_TCGEN05, pruned=A_pruned, vals=vals, meta=meta)
        if record:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        sp.gemm(vals, meta, Bt, alpha=cfg.alpha, beta=cfg.beta, C=C, out=Dout, cd=cd, ws=ws)  # Section 3.2
        if record:
            e1.record(stream)
            gemm_events.append((e0, e1))

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    D.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for _ in range(args.steps):
        step(record=True)
    t_end.record(stream)
    torch.cuda.synchronize()
    D.barrier()
    clocks = sampler.stop()
    elapsed_ms = D.max_over_ranks(t_begin.elapsed_time(t_end), dev)
    check_status("timed steps")
    gemm_ms = float(np.mean([a.elapsed_time(b) for a, b in gemm_events]))
    flop = cfg.dense_equiv_flop
    ms_per_step = elapsed_ms / args.steps
    value = world * flop / (ms_per_step * 1e-3) / 1e12

    # ---- per-kernel timings, dense variant (outside the timed region) ----
    def time_call(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            # keep the GPU busy while the host enqueues, so that the host's launch latency is not
            # part of the interval between the two events
            torch.cuda._sleep(400000)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.median(ts))

    es = 2 if ab != "i8" else 1
    prune_ms = time_call(lambda: sp.prune(A, out=A_pruned))
    compress_ms = time_call(lambda: sp.compress_into(A_pruned, vals, meta, layout=sp.META_TCGEN05))
    dense_ms = time_call(lambda: sp.gemm(A_pruned, None, Bt, alpha=cfg.alpha, beta=cfg.beta, C=C, out=Dout, cd=cd,
                                         a_is_dense=True, ws=ws), reps=3)
    fused_ms = time_call(lambda: sp.prune_compress(A, layout=sp.META_TCGEN05, pruned=A_pruned, vals=vals, meta=meta))
    prune_bytes = 2 * M * K * es
    compress_bytes = M * K * es + M * K // 2 * es + M * K // 8
    peaks = measured_peaks()
    sparse_peak = 2.0 * peaks["bf16_tflops"] * (2.0 if ab == "i8" else 1.0)
    gemm_tflops = flop / (gemm_ms * 1e-3) / 1e12
    kernels = {
        "prune_ms": prune_ms, "prune_gbs": prune_bytes / prune_ms / 1e6,
        "prune_frac_of_hbm_" + peaks["source"]: prune_bytes / prune_ms / 1e6 / peaks["hbm_gbs"],
        "compress_ms": compress_ms, "compress_gbs": compress_bytes / compress_ms / 1e6,
        "compress_frac_of_hbm_" + peaks["source"]: compress_bytes / compress_ms / 1e6 / peaks["hbm_gbs"],
        "prune_compress_fused_ms": fused_ms, "prune_compress_fused_gbs": (prune_bytes + compress_bytes - M * K * es) / fused_ms / 1e6,
        "prune_compress_fused_frac_of_hbm_" + peaks["source"]:
            (prune_bytes + compress_bytes - M * K * es) / fused_ms / 1e6 / peaks["hbm_gbs"],
        "gemm_ms": gemm_ms, "gemm_dense_equiv_tflops": gemm_tflops, "gemm_useful_tflops": gemm_tflops / 2,
        "gemm_frac_of_nominal_sparse_peak": gemm_tflops / (NOMINAL_SPARSE_BF16_TFLOPS * (2.0 if ab == "i8" else 1.0)),
        "dense_variant_ms": dense_ms, "dense_variant_tflops": flop / (dense_ms * 1e-3) / 1e12,
        "speedup_vs_dense_variant": dense_ms / gemm_ms,
    }

    # ---- context: cuBLAS dense on the same pruned matrix (a library call, not part of the path) ----
    if ab != "i8":
        torch_ms = time_call(lambda: torch.matmul(A_pruned, Bt.t()), reps=3)
        kernels["context_torch_matmul_dense_ms"] = torch_ms
        kernels["context_torch_matmul_dense_tflops"] = flop / (torch_ms * 1e-3) / 1e12
        kernels["speedup_vs_torch_matmul_dense"] = torch_ms / gemm_ms
        kernels["speedup_vs_best_dense"] = min(dense_ms, torch_ms) / gemm_ms
    check_status("per-kernel timings")

    # ---- sustained figures: about a second of back-to-back launches, the regime in which the 1 kW power
    # cap, not the burst clock, sets the rate (the comparison the measured sustained peak belongs to) ----
    def time_sustained(fn, seconds=1.0):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        n = max(3, int(seconds * 1000.0 / max(a.elapsed_time(b), 1e-3)))
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    if world == 1 and not args.rows and not args.no_sustained:
        sus_sampler = ClockSampler(local_rank, period_s=0.01)
        sus_sampler.start()
        sus_ms = time_sustained(lambda: sp.gemm(vals, meta, Bt, alpha=cfg.alpha, beta=cfg.beta, C=C, out=Dout, cd=cd, ws=ws))
        sus_clocks = sus_sampler.stop()
        kernels["gemm_sustained_ms"] = sus_ms
        # the clock the power cap allowed during that loop, and the time re-based to 1 GHz: a figure that can
        # be compared between runs and boxes whose power and thermal state differ
        if sus_clocks.get("sm_mhz"):
            kernels["gemm_sustained_sm_mhz"] = sus_clocks["sm_mhz"]
            kernels["gemm_sustained_ms_x_sm_ghz"] = sus_ms * sus_clocks["sm_mhz"] / 1e3
            kernels["gemm_sustained_clock_reasons"] = sus_clocks["reasons"]
        kernels["gemm_sustained_dense_equiv_tflops"] = flop / (sus_ms * 1e-3) / 1e12
        kernels["gemm_sustained_frac_of_2x_measured_sustained_dense"] = \
            flop / (sus_ms * 1e-3) / 1e12 / (2.0 * peaks["bf16_tflops_sustained"] * (2.0 if ab == "i8" else 1.0))
        if ab != "i8":
            tsus_ms = time_sustained(lambda: torch.matmul(A_pruned, Bt.t()))
            kernels["context_torch_matmul_dense_sustained_ms"] = tsus_ms
            kernels["sustained_speedup_vs_torch_matmul_dense"] = tsus_ms / sus_ms

    check_status("sustained loops")

    # ---- the other configurations (GEMM only, L2 flushed between repetitions) ----
    others = {}
    if world == 1 and not args.no_other_configs and not args.rows:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        flush_words = flush.view(torch.int32)

        def time_flushed(fn, reps=7):
            fn()
            ts = []
            for _ in range(reps):
                # write a buffer larger than the L2, then read it back: the read leaves the L2 full of
                # CLEAN lines, so that the kernel under test does not also pay for the write-back of up
                # to 126 MB of dirty lines of the flush itself
                flush.zero_()
                flush_words.sum()
                # keep the GPU busy while the host enqueues, so that launch latency of these short
                # kernels is not part of the interval between the two events
                torch.cuda._sleep(400000)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            return float(np.median(ts))

        def host_call_us(oc, ovals, ometa, oB, oD, calls=400):
            """CPU time of one sp24_gemm call at the C ABI (a ctypes call with prebuilt arguments: validation,
            tile choice, cached tensor maps, kernel launch); the GPU drains afterwards.  Python's own
            marshalling in the binding is not part of it."""
            import ctypes as ct
            desc = sp.make_desc(oc.ab_type, oc.cd_type, oc.M, oc.N, oc.K, oc.K // 2, oc.K, oc.N, oc.N)
            al, be = sp._scalar(oc.ab_type, 1), sp._scalar(oc.ab_type, 0)
            argv = (ct.byref(desc), ct.byref(al), ct.c_void_p(ovals.data_ptr()), ct.c_void_p(ometa.data_ptr()),
                    ct.c_void_p(oB.data_ptr()), ct.byref(be), None, ct.c_void_p(oD.data_ptr()),
                    ct.c_void_p(ws.data_ptr()), ws.numel(), stream.cuda_stream)
            fn = sp.lib.sp24_gemm
            assert fn(*argv) == 0
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(calls):
                fn(*argv)
            dt = time.perf_counter() - t0
            torch.cuda.synchronize()
            return 1e6 * dt / calls

        for name in inputs.CONFIG_ORDER:
            oc = inputs.CONFIGS[name]
            if name == cfg.name:
                continue
            oA = dev_tensor(inputs.gen_A(oc), oc.ab_type)
            if oc.conv is not None:
                x = dev_tensor(inputs.gen_conv_input(oc), oc.ab_type)
                im2col_ms = time_flushed(lambda: sp.im2col_nhwc_3x3(x), reps=3)
                oB = sp.im2col_nhwc_3x3(x)
            else:
                im2col_ms = None
                oB = dev_tensor(inputs.gen_Bt(oc), oc.ab_type)
            ovals, ometa, _ = sp.compress(oA)
            opruned = sp.prune(oA)
            oD = torch.empty((oc.M, oc.N), dtype=tdt[oc.cd_type], device=dev)
            s_ms = time_flushed(lambda: sp.gemm(ovals, ometa, oB, out=oD, cd=oc.cd_type, ws=ws))
            warm_ms = time_call(lambda: sp.gemm(ovals, ometa, oB, out=oD, cd=oc.cd_type, ws=ws))  # operands in the L2
            d_ms = time_flushed(lambda: sp.gemm(opruned, None, oB, out=oD, cd=oc.cd_type, a_is_dense=True, ws=ws))
            peak = 2.0 * peaks["bf16_tflops"] * (2.0 if oc.ab_type == "i8" else 1.0)
            nominal = NOMINAL_SPARSE_BF16_TFLOPS * (2.0 if oc.ab_type == "i8" else 1.0)
            odesc = sp.make_desc(oc.ab_type, oc.cd_type, oc.M, oc.N, oc.K, oc.K // 2, oc.K, oc.N, oc.N)
            others[name] = {"M": oc.M, "N": oc.N, "K": oc.K, "ab": oc.ab_type, "tile": sp.gemm_plan(odesc),
                            "gemm_ms": s_ms, "gemm_l2_warm_ms": warm_ms,
                            "frac_of_nominal_sparse_peak": oc.dense_equiv_flop / (s_ms * 1e-3) / 1e12 / nominal,
                            "host_call_us": host_call_us(oc, ovals, ometa, oB, oD),
                            "gemm_dense_equiv_tflops": oc.dense_equiv_flop / (s_ms * 1e-3) / 1e12,
                            "frac_of_2x_measured_dense": oc.dense_equiv_flop / (s_ms * 1e-3) / 1e12 / peak,
                            "dense_variant_ms": d_ms, "speedup_vs_dense_variant": d_ms / s_ms}
            if im2col_ms is not None:
                others[name]["im2col_ms"] = im2col_ms
                oD2 = torch.empty((oc.M, oc.N), dtype=tdt[oc.cd_type], device=dev)
                c_ms = time_flushed(lambda: sp.conv3x3_nhwc(ovals, ometa, x, out=oD2, cd=oc.cd_type, ws=ws))
                others[name]["implicit_conv_ms"] = c_ms
                others[name]["implicit_conv_dense_equiv_tflops"] = oc.dense_equiv_flop / (c_ms * 1e-3) / 1e12
                del oD2
            if oc.ab_type == "i8":
                # the dequantising epilogue (per-row scales) with bf16 and int8 outputs
                rs = torch.full((oc.M,), 1e-5, dtype=torch.float32, device=dev)
                for out_t in ("bf16", "i8"):
                    oQ = torch.empty((oc.M, oc.N), dtype=tdt[out_t], device=dev)
                    q_ms = time_flushed(lambda: sp.gemm_i8_dequant(ovals, ometa, oB, rs, cd=out_t, out_scale=0.05,
                                                                   out=oQ, ws=ws))
                    others[name][f"dequant_{out_t}_ms"] = q_ms
                    others[name][f"dequant_{out_t}_dense_equiv_tflops"] = oc.dense_equiv_flop / (q_ms * 1e-3) / 1e12
                    del oQ
            del oA, oB, ovals, ometa, opruned, oD
        # TF32 mode with the 1:2 pattern (Section 3.2, Table 1) on a 4096 x 8192 x 4096 problem
        tA = (torch.randn(4096, 4096, device=dev) * 0.02)
        tB = torch.randn(8192, 4096, device=dev)
        tvals, tmeta, _ = sp.compress(tA)
        tprun = sp.prune(tA)
        tD = torch.empty((4096, 8192), dtype=torch.float32, device=dev)
        t_s = time_flushed(lambda: sp.gemm(tvals, tmeta, tB, out=tD, ws=ws))
        t_d = time_flushed(lambda: sp.gemm(tprun, None, tB, out=tD, a_is_dense=True, ws=ws))
        tflop = 2.0 * 4096 * 8192 * 4096
        others["tf32_1of2_4096x8192x4096"] = {
            "gemm_ms": t_s, "gemm_dense_equiv_tflops": tflop / (t_s * 1e-3) / 1e12,
            "frac_of_measured_dense_bf16": tflop / (t_s * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "dense_variant_ms": t_d, "speedup_vs_dense_variant": t_d / t_s}
        del tA, tB, tvals, tmeta, tprun, tD
        # 8-bit floating-point operands (e4m3; not in the paper's Table 1) on a 16384 x 8192 x 8192 problem
        fA = (torch.randn(16384, 8192, device=dev)).to(torch.float8_e4m3fn)
        fB = torch.randn(8192, 8192, device=dev).to(torch.float8_e4m3fn)
        fvals, fmeta, _ = sp.compress(fA)
        fprun = sp.prune(fA)
        fD = torch.empty((16384, 8192), dtype=torch.bfloat16, device=dev)
        f_s = time_flushed(lambda: sp.gemm(fvals, fmeta, fB, out=fD, cd="bf16", ws=ws))
        f_d = time_flushed(lambda: sp.gemm(fprun, None, fB, out=fD, cd="bf16", a_is_dense=True, ws=ws))
        fflop = 2.0 * 16384 * 8192 * 8192
        others["fp8_e4m3_16384x8192x8192"] = {
            "gemm_ms": f_s, "gemm_dense_equiv_tflops": fflop / (f_s * 1e-3) / 1e12,
            "frac_of_2x_measured_dense": fflop / (f_s * 1e-3) / 1e12 / (4.0 * peaks["bf16_tflops"]),
            "dense_variant_ms": f_d, "speedup_vs_dense_variant": f_d / f_s}
        del fA, fB, fvals, fmeta, fprun, fD
        # FP16 accumulation (Table 1's FP16-accumulate row) against FP32 accumulation, same kernel and shape
        hA = (torch.randn(16384, 8192, device=dev) * 0.02).half()
        hB = torch.randn(8192, 8192, device=dev).half()
        hvals, hmeta, _ = sp.compress(hA)
        hD = torch.empty((16384, 8192), dtype=torch.float16, device=dev)
        h32 = time_flushed(lambda: sp.gemm(hvals, hmeta, hB, out=hD, cd="f16", ws=ws))
        h16 = time_flushed(lambda: sp.gemm(hvals, hmeta, hB, out=hD, cd="f16", ws=ws, acc_f16=True))
        hflop = 2.0 * 16384 * 8192 * 8192
        others["f16_accumulate_16384x8192x8192"] = {
            "fp32_accumulate_ms": h32, "fp16_accumulate_ms": h16, "fp16_over_fp32_time": h16 / h32,
            "fp16_accumulate_dense_equiv_tflops": hflop / (h16 * 1e-3) / 1e12}
        del flush, flush_words, hA, hB, hvals, hmeta, hD
        check_status("other configurations")

    # ---- end to end through the host-buffer entry point (rank-local) ----
    import ctypes
    e2e = None
    e2e_steps = 0 if args.no_e2e else max(1, min(args.steps, 3))
    if e2e_steps:
        hA = torch.from_numpy(A_h.view(np.int16) if es == 2 else A_h).pin_memory()
        hB = torch.from_numpy(Bt_h.view(np.int16) if es == 2 else Bt_h).pin_memory()
        hC = torch.from_numpy(C_h.view(np.int16) if cd in ("f16", "bf16") else C_h).pin_memory() if C_h is not None else None
        hD = torch.empty((M, N), dtype=torch.int16 if cd in ("f16", "bf16") else tdt[cd]).pin_memory()
        desc = sp.make_desc(ab, cd, M, N, K, K // 2, K, N, N)
        al, be = sp._scalar(ab, cfg.alpha), sp._scalar(ab, cfg.beta)
        vp = lambda t: ctypes.c_void_p(t.data_ptr()) if t is not None else None  # noqa: E731

        def e2e_step():
            st = sp.lib.sp24_pipeline_host(ctypes.byref(desc), ctypes.byref(al), vp(hA), vp(hB), ctypes.byref(be), vp(hC),
                                           vp(hD), vp(A_pruned), vp(vals), vp(meta), vp(Bt), vp(C), vp(Dout), vp(ws),
                                           ws.numel(), stream.cuda_stream)
            if st != 0:
                raise SystemExit(f"sp24_pipeline_host: {sp.status_string(st)}")

        e2e_step()
        torch.cuda.synchronize()
        D.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        b.record(stream)
        torch.cuda.synchronize()
        e2e_ms = D.max_over_ranks(a.elapsed_time(b), dev) / e2e_steps
        h2d = A_h.nbytes + Bt_h.nbytes + (C_h.nbytes if C_h is not None else 0)
        d2h = M * N * (2 if cd in ("f16", "bf16") else 4)
        e2e = {"value": world * flop / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps}

    if rank != 0:
        return
    tile = sp.gemm_plan(sp.make_desc(ab, cd, M, N, K, K // 2, K, N, N))
    tc, tn, tm = (int(v) for v in tile.split("x"))
    kernel_name = (f"sp24_gemm (tcgen05.mma.sp, {'CTA pairs' if tc == 2 else 'single CTAs'}, "
                   f"{128 * tc * tm}x{tn} tiles)")
    nominal_peak = NOMINAL_SPARSE_BF16_TFLOPS * (2.0 if ab == "i8" else 1.0)
    roofline = {
        "kernel": kernel_name, "bound": "tensor", "achieved": gemm_tflops, "peak": sparse_peak, "unit": UNIT,
        "frac": gemm_tflops / sparse_peak,
        "peak_source": f"2 x {peaks['source']} dense bf16 burst ({peaks['bf16_tflops']} TFLOP/s)"
                       + (" x 2 for int8" if ab == "i8" else ""),
        "frac_of_2x_sustained": (gemm_tflops / (2.0 * peaks["bf16_tflops_sustained"])
                                 if peaks.get("bf16_tflops_sustained") and ab != "i8" else None),
        "nominal_peak": nominal_peak, "frac_of_nominal": gemm_tflops / nominal_peak,
        "target": "north_star asks for >= 0.70 of the sparse tensor peak and >= 1.5x the dense variant",
        "target_met": {"frac_of_measured_peak": gemm_tflops / sparse_peak >= 0.70,
                       "frac_of_nominal_peak": gemm_tflops / nominal_peak >= 0.70,
                       "speedup_vs_dense_variant": kernels["speedup_vs_dense_variant"] >= 1.5,
                       "speedup_vs_best_dense": kernels.get("speedup_vs_best_dense", 0.0) >= 1.5},
        "traffic": ncu_traffic("sp24_gemm", cfg.name),
    }
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        v, sample, threads = oracle_sample(cfg, 15.0)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if ab == "bf16" else ("f16" if ab == "f16" else "i8"), "data": "synthetic",
        "config": {"workload": cfg.name, "M": M, "N": N, "K": K, "alpha": cfg.alpha, "beta": cfg.beta,
                   "cd_type": cd, "tokens_per_gpu": N, "parallelism": f"replicated weight, tokens sharded x{world}",
                   "l2": "inputs larger than L2 (A 1.2 GB, vals 0.6 GB, B 0.2 GB per step)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 2 * args.steps, "roofline": roofline, "cpu_baseline": cpu,
        "kernels": kernels, "other_configs": others,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="gpt3_ffn_bf16", choices=inputs.CONFIG_ORDER)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the GEMM timings of the other configurations")
    ap.add_argument("--no-sustained", action="store_true", help="skip the one-second sustained GEMM loops")
    ap.add_argument("--rows", type=int, default=0,
                    help="use only the first ROWS rows of A (a smaller case of the same kernel for ncu captures)")
    args = ap.parse_args()
    cfg = inputs.CONFIGS[args.config]
    if args.rows:
        cfg = inputs.scaled(cfg, M=args.rows, name=f"{cfg.name}[rows={args.rows} of {cfg.M}]")
    if cfg.conv is not None:
        raise SystemExit("the convolution config is covered by the parity tests, not by bench.py")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
