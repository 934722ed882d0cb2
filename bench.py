#!/usr/bin/env python
"""Benchmark of the Qift quantized-linear hot path on B200.

Default arm: one "step" = one decode token (M = 1) through the 7 linear shapes of a LLaMA-2-7B
layer, for 32 layers of distinct synthetic weights (224 modules, 1.63 GB of packed weights, so every
step streams far more than the 126 MB L2).  Each module runs the whole path through the C ABI:
rotate + INT4-quantize the activation row, then the exact W2A4 product and scale epilogue.  The
metric is algorithmic HBM bytes per second; `roofline` times the product kernel alone over the same
224 weight matrices; `prefill` reports the M = 2048 tcgen05 GEMM on LLaMA-3.1-8B shapes in TOPS;
`e2e` runs the same step through the host-buffer entry point with the copies inside the timed
region; `cpu_baseline` times the CPU oracle on a bounded sample.

`--impl reference` times the CPU oracle (a deliberately plain single-threaded program) instead.

Launch: python bench.py --gpus N --steps K --warmup W   (N > 1 under torch.distributed.run:
independent replicas, one per GPU, weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synth  # noqa: E402

CLIP = 0.9
N_LAYERS = 32
# dram__bytes_read.sum + dram__bytes_write.sum of one linear_grouped_kernel launch in the ncu capture of
# the 4-layer case (profiles/linear_grouped_kernel_llama2_m1_4layers.md): 203 236 864 + 4 653 056 bytes
# for 203 877 488 algorithmic bytes.  Every packed word is read once, so traffic scales with the layers.
NCU_TRAFFIC_BYTES_4_LAYERS = 207318528   # dram__bytes_read.sum + dram__bytes_write.sum of linear_grouped_kernel, 4-layer capture (profiles/)


# ------------------------------------------------------------------------------------------------
# algorithmic bytes / ops (per module call)
# ------------------------------------------------------------------------------------------------
def product_bytes(M, N, K, bits=2, out_bytes=4):
    """Packed codes + channel scales + int8 activations and token scales + output."""
    return N * K * bits // 8 + 4 * N + M * (K + 4) + M * N * out_bytes


def quant_bytes(M, K, in_bytes=4):
    """Activation row read + int8 row and scale written."""
    return M * K * in_bytes + M * K + 4 * M


def reduce_max_ms(dist, ms, device):
    """Step time of the job = the slowest rank's (device-measured) time."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(world, bytes_per_rank, ms_per_step):
    """Whole-job GB/s: every replica moves bytes_per_rank per step, in ms_per_step."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# clocks sampling during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
class Module:
    __slots__ = ("name", "N", "K", "B", "packed", "s_n", "x", "y", "x_host", "y_host", "bits", "levels", "levels_i8")


def build_stack(torch, qift, shapes, n_layers, M, levels_of_layer, seed, x_dtype, y_dtype, device, gen):
    """Synthetic stack: Student-t(5)*0.02 weights rotated by the blockwise Hadamard (our kernel),
    MSE-scaled and packed (our kernel); Gaussian activations with 1% outlier channels x20."""
    mods = []
    for layer in range(n_layers):
        lv = levels_of_layer(layer)
        for (name, N, K) in shapes:
            z = torch.randn((N, K), device=device, dtype=torch.float32, generator=gen)
            chi = torch.zeros((N, K), device=device, dtype=torch.float32)
            for _ in range(5):
                chi += torch.randn((N, K), device=device, dtype=torch.float32, generator=gen) ** 2
            W = 0.02 * z / torch.sqrt(chi / 5.0)
            del z, chi
            B = synth.had_block_for(K)
            qift.qift_rotate(W, B, out=W)
            m = Module()
            m.name, m.N, m.K, m.B, m.levels = name, N, K, B, lv
            m.bits = 4 if lv == qift.INT4 else 2
            m.packed, m.s_n = qift.qift_pack_weights(W, lv, qift.SCALE_MSE)
            del W
            x = torch.randn((M, K), device=device, dtype=torch.float32, generator=gen)
            n_out = max(1, round(0.01 * K))
            ch = torch.randperm(K, device=device, generator=gen)[:n_out]
            x[:, ch] *= 20.0
            m.x = x.to(x_dtype).contiguous()
            m.y = torch.empty((M, N), device=device, dtype=y_dtype)
            m.x_host = m.x.cpu().pin_memory()
            m.y_host = torch.empty((M, N), dtype=y_dtype).pin_memory()
            mods.append(m)
    torch.cuda.synchronize()
    return mods


def run_gpu(args):
    import torch

    import paper_2606_02823_b200 as qift

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)
    L = qift.lib()
    gen = torch.Generator(device=device)
    gen.manual_seed(2000 + rank)
    M = 1
    launches = [0]

    mods = build_stack(torch, qift, synth.LLAMA2_7B, args.layers, M, lambda l: qift.MNZ, 2000, torch.float32, torch.float32,
                       device, gen)
    kmax = max(m.K for m in mods)
    q_a = torch.empty((M, kmax), dtype=torch.int8, device=device)
    s_a = torch.empty((M,), dtype=torch.float32, device=device)
    vp = ctypes.c_void_p

    def check(rc):
        if rc != 0:
            raise RuntimeError(f"qift call failed: {qift.status_string(rc)}")

    def step_full(stream):
        st = vp(stream)
        for m in mods:
            check(L.qift_quantize_act(vp(m.x.data_ptr()), qift.F32, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st))
            check(L.qift_w2a4_linear(vp(m.packed.data_ptr()), vp(m.s_n.data_ptr()), m.levels, vp(q_a.data_ptr()),
                                     vp(s_a.data_ptr()), M, m.N, m.K, vp(m.y.data_ptr()), qift.F32, None, None, 0, st))
        return 2 * len(mods)

    def step_product_only(stream):
        st = vp(stream)
        for m in mods:
            check(L.qift_w2a4_linear(vp(m.packed.data_ptr()), vp(m.s_n.data_ptr()), m.levels, vp(q_a.data_ptr()),
                                     vp(s_a.data_ptr()), M, m.N, m.K, vp(m.y.data_ptr()), qift.F32, None, None, 0, st))
        return len(mods)

    scratch_bytes = max(qift.qift_forward_scratch_bytes(M, m.N, m.K, m.levels, qift.F32, qift.F32) for m in mods)
    scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=device)

    def step_host(stream):
        st = vp(stream)
        for m in mods:
            check(L.qift_forward_host(vp(m.x_host.data_ptr()), qift.F32, M, m.K, m.B, CLIP, vp(m.packed.data_ptr()),
                                      vp(m.s_n.data_ptr()), m.levels, m.N, vp(m.y_host.data_ptr()), qift.F32,
                                      vp(scratch.data_ptr()), scratch_bytes, st))

    # grouped path: the whole step as one plan (one quantizer launch + one persistent product launch)
    plan = qift.qift_group_plan([(m.x, m.packed, m.s_n, m.B) for m in mods], qift.MNZ, CLIP, arenas=True)
    ph, pd = vp(plan.host.data_ptr()), vp(plan.dev.data_ptr())
    x_bytes, y_bytes = plan.x_arena.numel(), plan.y_arena.numel()

    def step_grouped_host(stream):
        check(L.qift_group_forward_host(ph, pd, vp(plan.x_host.data_ptr()), vp(plan.x_arena.data_ptr()), x_bytes,
                                        vp(plan.y_arena.data_ptr()), vp(plan.y_host.data_ptr()), y_bytes, vp(stream)))

    def step_grouped(stream):
        check(L.qift_group_forward(ph, pd, vp(stream)))
        return 2

    def step_grouped_product(stream):
        check(L.qift_group_linear(ph, pd, vp(stream)))
        return 1

    def capture(fn):
        """Capture one step into a CUDA graph (programmatic-dependent-launch edges included)."""
        side = torch.cuda.Stream(device=device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn(side.cuda_stream)   # warm-up outside capture: attribute calls, lazy module load
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(g, stream=side):
                n = fn(torch.cuda.current_stream().cuda_stream)
            return g, n
        except Exception as e:  # noqa: BLE001
            sys.stderr.write(f"bench: graph capture failed ({e}); timing direct launches\n")
            return None, fn(torch.cuda.current_stream().cuda_stream)

    def timed(run_once, steps, warmup):
        for _ in range(warmup):
            run_once()
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            run_once()
        e1.record()
        torch.cuda.synchronize()
        ms = reduce_max_ms(dist, e0.elapsed_time(e1), device)
        if dist:
            dist.barrier()
        return ms

    stream = torch.cuda.current_stream()
    g_full, n_full = capture(step_full)
    g_prod, n_prod = capture(step_product_only)
    run_full = (lambda: g_full.replay()) if g_full else (lambda: step_full(stream.cuda_stream))
    run_prod = (lambda: g_prod.replay()) if g_prod else (lambda: step_product_only(stream.cuda_stream))
    step_grouped(stream.cuda_stream)
    torch.cuda.synchronize()
    run_grp = lambda: step_grouped(stream.cuda_stream)
    run_grp_prod = lambda: step_grouped_product(stream.cuda_stream)

    bytes_product = sum(product_bytes(M, m.N, m.K, m.bits) for m in mods)
    bytes_step = bytes_product + sum(quant_bytes(M, m.K) for m in mods)

    # the clock sampler runs across every timed region below (the headline loop alone lasts tens of
    # milliseconds, shorter than one nvidia-smi sampling period)
    sampler = ClockSampler(local)
    sampler.start()
    ms_grp = timed(run_grp, args.steps, args.warmup)
    ms_grp_prod = timed(run_grp_prod, args.steps, args.warmup)
    pc_steps = max(3, min(args.steps, 50))
    ms_full = timed(run_full, pc_steps, args.warmup)
    ms_prod = timed(run_prod, pc_steps, args.warmup)

    # end to end: host buffers in, host buffers out, copies inside the timed region
    def run_host():
        step_grouped_host(stream.cuda_stream)
        stream.synchronize()
    e2e_steps = max(3, min(args.steps, 100))
    ms_host = timed(run_host, e2e_steps, 3)

    # the same step as four plans of a quarter of the modules each, alternating between two streams: the copies
    # of one chunk overlap the kernels of the other (one call per chunk, same entry point)
    n_chunks = max(1, min(4, len(mods) // 7))   # measured: 2 / 4 / 8 / 16 chunks -> 0.376 / 0.358 / 0.390 / 0.535 ms per step
    per = (len(mods) + n_chunks - 1) // n_chunks
    chunk_plans = [qift.qift_group_plan([(m.x, m.packed, m.s_n, m.B) for m in mods[i * per:(i + 1) * per]], qift.MNZ, CLIP,
                                        arenas=True) for i in range(n_chunks)]
    torch.cuda.synchronize()
    side = [torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)]

    def run_host_chunked():
        for i, cp in enumerate(chunk_plans):
            check(L.qift_group_forward_host(vp(cp.host.data_ptr()), vp(cp.dev.data_ptr()), vp(cp.x_host.data_ptr()),
                                            vp(cp.x_arena.data_ptr()), cp.x_arena.numel(), vp(cp.y_arena.data_ptr()),
                                            vp(cp.y_host.data_ptr()), cp.y_arena.numel(), vp(side[i % 2].cuda_stream)))
        side[0].synchronize()
        side[1].synchronize()
    ms_host_chunked = timed(run_host_chunked, e2e_steps, 3)

    def run_host_percall():
        step_host(stream.cuda_stream)
        stream.synchronize()
    ms_host_pc = timed(run_host_percall, 5, 2)
    for _ in range(3):      # keep the GPU under the same load until the sampler has a few readings
        ms_grp_again = timed(run_grp, args.steps, 0)
    clocks = sampler.stop()
    rc, detail = qift.qift_device_status()
    if rc != 0:
        raise RuntimeError(f"device status {rc} detail {detail:#x}")

    pk = peaks()
    step_ms = ms_grp / args.steps
    value = aggregate_throughput(world, bytes_step, step_ms)
    launch_us = ms_grp_prod / args.steps * 1e3          # one persistent launch per step
    achieved = bytes_product / (launch_us * 1e-6) / 1e9
    percall_ms = ms_full / pc_steps
    percall_prod_us = ms_prod / pc_steps * 1e3 / n_prod
    host_ms = ms_host_chunked / e2e_steps
    host_single_ms = ms_host / e2e_steps
    out = {
        "metric": "w2a4_decode_hbm_gbs", "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(step_ms, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": "config 2: LLaMA-2-7B-shaped decode, M=1, 7 linear shapes x 32 layers of distinct weights, "
                               "MNZ {+-1,+-3}, Hadamard + INT4 act quant + W2A4 product per module, grouped API (2 launches per step)" +
                               ("" if args.layers == N_LAYERS else f" [REDUCED to {args.layers} layers: not a bench number]"),
                   "tokens_per_step": M, "modules_per_step": len(mods), "packed_weight_bytes": sum(m.packed.numel() * 4 for m in mods),
                   "l2": f"inputs larger than L2: each step streams {sum(m.packed.numel() * 4 for m in mods) / 1e9:.2f} GB of distinct packed weights",
                   "cuda_graph": False, "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "tokens_per_s": round(world * M / (step_ms * 1e-3), 1),
        "pct_of_8TBs": round(100 * value / world / 8000.0, 2),
        "roofline": {"bound": "hbm", "kernel": "linear_grouped_kernel", "achieved": round(achieved, 1), "peak": pk["hbm_gbs"],
                     "unit": "GB/s", "frac": round(achieved / pk["hbm_gbs"], 4),
                     "traffic": round(NCU_TRAFFIC_BYTES_4_LAYERS * args.layers / 4),
                     "traffic_source": "ncu capture of the 4-layer case, scaled by layers",
                     "peak_source": pk["source"], "avg_launch_us": round(launch_us, 3),
                     "algorithmic_bytes_per_launch": bytes_product},
        "per_call": {"what": "same step as 224 x (qift_quantize_act + qift_w2a4_linear) in one CUDA graph with "
                             "programmatic dependent launch", "value": round(world * bytes_step / (percall_ms * 1e-3) / 1e9, 2),
                     "unit": "GB/s", "ms_per_step": round(percall_ms, 5), "cuda_graph": g_full is not None,
                     "product_only_avg_launch_us": round(percall_prod_us, 3), "launches_per_step": n_full},
        "e2e": {"value": round(world * bytes_step / (host_ms * 1e-3) / 1e9, 2), "unit": "GB/s",
                "h2d_bytes_per_step": x_bytes, "d2h_bytes_per_step": y_bytes,
                "ms_per_step": round(host_ms, 4),
                "api": f"{n_chunks} x qift_group_forward_host (pinned host arenas in and out), one call per quarter of the "
                       "modules, alternating between two streams so that copies overlap kernels",
                "single_call": {"api": "1 x qift_group_forward_host on one stream", "ms_per_step": round(host_single_ms, 4),
                                "value": round(world * bytes_step / (host_single_ms * 1e-3) / 1e9, 2)},
                "per_call_api": {"api": "224 x qift_forward_host", "ms_per_step": round(ms_host_pc / 5, 4),
                                 "value": round(world * bytes_step / (ms_host_pc / 5 * 1e-3) / 1e9, 2)}},
        "gpu_launches": 2 * args.steps,
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_prefill:
        out["mixed_stack"] = run_mixed_stack(torch, qift, L, device, gen, args)
        out["batched_decode"] = run_batched_decode(torch, qift, L, device, gen, args)
        out["prefill"] = run_prefill(torch, qift, L, device, gen, pk)
        out["kv4"] = run_kv4(torch, qift, L, pk)
        out["diagnostics"] = run_diagnostics(torch, qift, pk)
    if rank == 0 and world == 1 and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline(budget_s=12.0)
    if rank == 0:
        print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


def run_mixed_stack(torch, qift, L, device, gen, args):
    """Config 5: layer-wise mixed precision on LLaMA-2-7B shapes at M = 1: the first L layers INT4 weights (W4A4), the
    rest MNZ (W2A4), b_avg = 2 + L/16 bits per weight for 32 layers (Sec. 3.7).  Config 5 itself is L = 16 (3 bits on
    average); the sweep adds L = 4, 8, 12.  Two grouped plans (a plan holds one level set): four launches per
    token-step.  Modules run on their own staged inputs, as in the headline."""
    vp = ctypes.c_void_p
    st = vp(torch.cuda.current_stream().cuda_stream)

    def point(n4, n2):
        plans, algo = [], 0
        for lv, n in ((qift.INT4, n4), (qift.MNZ, n2)):
            mods = build_stack(torch, qift, synth.LLAMA2_7B, n, 1, lambda l, lv=lv: lv, 5000 + lv, torch.float32, torch.float32,
                               device, gen)
            plans.append((qift.qift_group_plan([(m.x, m.packed, m.s_n, m.B) for m in mods], lv, CLIP), mods))
            algo += sum(product_bytes(1, m.N, m.K, m.bits) + quant_bytes(1, m.K) for m in mods)

        def step():
            for plan, _ in plans:
                rc = L.qift_group_forward(vp(plan.host.data_ptr()), vp(plan.dev.data_ptr()), st)
                assert rc == 0, rc

        for _ in range(5):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        steps = max(3, min(args.steps, 100))
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        return {"w4_layers": n4, "w2_layers": n2, "bits_per_weight": round(2 + 2 * n4 / (n4 + n2), 3), "ms_per_step": round(ms, 5),
                "tokens_per_s": round(1.0 / (ms * 1e-3), 1), "value": round(algo / (ms * 1e-3) / 1e9, 2), "unit": "GB/s",
                "algorithmic_bytes_per_step": algo, "pct_of_8TBs": round(100 * algo / (ms * 1e-3) / 8e12, 2)}

    n4 = max(1, args.layers // 2)
    out = point(n4, max(1, args.layers - n4))
    out["workload"] = (f"config 5: {out['w4_layers']} W4A4 layers + {out['w2_layers']} W2A4 (MNZ) layers, LLaMA-2-7B shapes, M=1, "
                       "grouped API (4 launches per step)")
    if args.layers >= 16:
        out["l_sweep"] = [point(args.layers * l // 32, args.layers - args.layers * l // 32) for l in (4, 8, 12)]
    out["prefill_m2048"] = mixed_prefill(torch, qift, L, device, gen, args, n4)
    return out


def mixed_prefill(torch, qift, L, device, gen, args, n4):
    """Config 5 at M = 2048: the same mixed stack (first layers W4A4, the rest W2A4 MNZ), every module as activation
    quantizer + product through the per-call API (bf16 in, bf16 out; AUTO route = codes expanded into one shared int8
    scratch, then the CTA-pair tcgen05 GEMM).  Distinct weights per layer; end-to-end linear-stack tokens per second."""
    M = 2048
    vp = ctypes.c_void_p
    st = vp(torch.cuda.current_stream().cuda_stream)
    mods = build_stack(torch, qift, synth.LLAMA2_7B, args.layers, M, lambda l: qift.INT4 if l < n4 else qift.MNZ, 5100,
                       torch.bfloat16, torch.bfloat16, device, gen)
    kmax = max(m.K for m in mods)
    q_a = torch.empty((M, kmax), dtype=torch.int8, device=device)
    s_a = torch.empty((M,), dtype=torch.float32, device=device)
    ws_bytes = max(qift.qift_workspace_bytes(M, m.N, m.K, m.levels) for m in mods)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=device)

    def step():
        for m in mods:
            rc = L.qift_quantize_act(vp(m.x.data_ptr()), qift.BF16, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st)
            assert rc == 0, rc
            fn = L.qift_w4a4_linear if m.levels == qift.INT4 else None
            if fn is not None:
                rc = fn(vp(m.packed.data_ptr()), vp(m.s_n.data_ptr()), vp(q_a.data_ptr()), vp(s_a.data_ptr()), M, m.N, m.K,
                        vp(m.y.data_ptr()), qift.BF16, None, vp(ws.data_ptr()), ws_bytes, st)
            else:
                rc = L.qift_w2a4_linear(vp(m.packed.data_ptr()), vp(m.s_n.data_ptr()), m.levels, vp(q_a.data_ptr()),
                                        vp(s_a.data_ptr()), M, m.N, m.K, vp(m.y.data_ptr()), qift.BF16, None, vp(ws.data_ptr()),
                                        ws_bytes, st)
            assert rc == 0, rc

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 3
    ops = 2.0 * M * sum(m.N * m.K for m in mods)
    return {"workload": f"config 5 at M = 2048: {n4} W4A4 + {args.layers - n4} W2A4 layers, LLaMA-2-7B shapes, per-call API with "
                        "activation quantizer", "ms_per_step": round(ms, 3), "tokens_per_s": round(M / (ms * 1e-3), 1),
            "tops": round(ops / (ms * 1e-3) / 1e12, 1), "launches_per_step": 3 * len(mods)}


def run_batched_decode(torch, qift, L, device, gen, args):
    """Config 3: LLaMA-3.1-8B shapes, batched decode at M = 1, 4, 16 token rows, PoT {+-1,+-4} against the standard
    {-2,-1,0,+1} set; grouped API (2 launches per step), 16 layers of distinct weights (0.87 GB per level set, larger
    than L2), every module on its own activation.  Bytes = packed weights + scales + activations + outputs."""
    vp = ctypes.c_void_p
    st = vp(torch.cuda.current_stream().cuda_stream)
    layers = max(1, min(16, args.layers))
    rows = []
    for name, lv in (("PoT", qift.POT), ("SYM", qift.SYM)):
        base = build_stack(torch, qift, synth.LLAMA31_8B, layers, 16, lambda l, lv=lv: lv, 6000 + lv, torch.float32, torch.float32,
                           device, gen)
        for M in (1, 4, 16):
            plan = qift.qift_group_plan([(m.x[:M].contiguous(), m.packed, m.s_n, m.B) for m in base], lv, CLIP)
            algo = sum(product_bytes(M, m.N, m.K, m.bits) + quant_bytes(M, m.K) for m in base)

            def step():
                rc = L.qift_group_forward(vp(plan.host.data_ptr()), vp(plan.dev.data_ptr()), st)
                assert rc == 0, rc

            for _ in range(5):
                step()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            steps = max(3, min(args.steps, 100))
            e0.record()
            for _ in range(steps):
                step()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / steps
            rows.append({"levels": name, "M": M, "ms_per_step": round(ms, 5), "tokens_per_s": round(M / (ms * 1e-3), 1),
                         "value": round(algo / (ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                         "pct_of_8TBs": round(100 * algo / (ms * 1e-3) / 8e12, 1)})
            del plan
        del base
    return {"workload": f"config 3: LLaMA-3.1-8B shapes, {layers} layers, grouped API, whole step (quantizer + product)", "points": rows}


def run_kv4(torch, qift, L, pk):
    """KV4 cache path: decode attention over a 4-bit cache (LLaMA-3.1-8B heads: 32 query / 8 KV heads of 128, 32768
    cached tokens, 32 layers of distinct caches = 1.2 GB) and the cache quantizer.  Bytes = codes + scales + zero-points."""
    vp = ctypes.c_void_p
    T, Hq, Hkv, D, layers = 32768, 32, 8, 128, 32
    caches = []
    for _ in range(layers):
        K, V = qift.Kv4Cache(Hkv, T), qift.Kv4Cache(Hkv, T, qift.KV_VALUES)
        for c in (K, V):
            c.codes.random_(0, 256)
            c.scale.uniform_(0.05, 0.2)
            c.zero.random_(0, 16)
        caches.append((K, V))
    q = torch.randn(Hq, D, device="cuda")
    o = torch.empty(Hq, D, device="cuda")
    ws = torch.empty(qift.qift_kv4_attention_workspace_bytes(T, Hq, Hkv), dtype=torch.uint8, device="cuda")
    st = vp(torch.cuda.current_stream().cuda_stream)

    def step():
        for K, V in caches:
            rc = L.qift_kv4_attention_decode(vp(q.data_ptr()), vp(K.codes.data_ptr()), vp(K.scale.data_ptr()), vp(K.zero.data_ptr()),
                                             vp(V.codes.data_ptr()), vp(V.scale.data_ptr()), vp(V.zero.data_ptr()), T, T, Hq, Hkv, D,
                                             vp(o.data_ptr()), vp(ws.data_ptr()), ws.numel(), st)
            assert rc == 0, rc

    def timed(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    ms = timed(step, 5)
    cache_bytes = layers * 2 * Hkv * T * (D // 2 + 8)
    gbs = cache_bytes / (ms * 1e-3) / 1e9
    # quantizer: 8192 new tokens of all 8 KV heads (bf16 in), with the head-dimension rotation
    x = torch.randn(8192, Hkv, D, device="cuda", dtype=torch.bfloat16)
    Kq = qift.Kv4Cache(Hkv, 8192)

    def quant():
        rc = L.qift_kv4_quantize(vp(x.data_ptr()), qift.BF16, 8192, Hkv, D, D, ctypes.c_float(0.95), 0, 8192, qift.KV_KEYS,
                                 vp(Kq.codes.data_ptr()), vp(Kq.scale.data_ptr()), vp(Kq.zero.data_ptr()), st)
        assert rc == 0, rc

    msq = timed(quant, 20)
    qbytes = 8192 * Hkv * (2 * D + D // 2 + 8)
    return {"workload": f"decode attention over a KV4 cache: {Hq} query / {Hkv} KV heads x {D}, {T} cached tokens, {layers} layers of "
                        "distinct caches (two launches per layer)", "us_per_layer": round(ms * 1e3 / layers, 2),
            "value": round(gbs, 1), "unit": "GB/s", "algorithmic_bytes_per_layer": cache_bytes // layers,
            "roofline": {"bound": "hbm", "kernel": "kv4_attention_partial_kernel", "achieved": round(gbs, 1), "peak": pk["hbm_gbs"],
                         "unit": "GB/s", "frac": round(gbs / pk["hbm_gbs"], 4),
                         "note": "both products on mma.sync fp16 with fp32 accumulators; the unpacking of the codes into operand "
                                 "registers keeps it instruction-bound above its memory time"},
            "quantizer": {"workload": "8192 tokens x 8 heads x 128, bf16 in, Hadamard over the head dimension", "us": round(msq * 1e3, 2),
                          "value": round(qbytes / (msq * 1e-3) / 1e9, 1), "unit": "GB/s"}}


def run_diagnostics(torch, qift, pk):
    """Quantizer diagnostics (Sec. 4.5): bucket statistics of one LLaMA-2 gate matrix (11008 x 4096 synthetic rotated
    weights, 225 MB of weights + codes), the float-grid quantizer with its 80-candidate sweep on the same matrix, and the
    ratio scan at the paper's size (100 000 pooled samples, the 0.005 grid of 199 ratios)."""
    N, K = 11008, 4096
    W = torch.randn(N, K, device="cuda") * 0.02
    lloyd = [-1.5104, -0.4528, 0.4528, 1.5104]
    s, codes = qift.qift_diag_grid_quantize(W, lloyd, qift.SCALE_MSE)

    def timed(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    ms_q = timed(lambda: qift.qift_diag_grid_quantize(W, lloyd, qift.SCALE_MSE, s_n=s), 3)
    ms_b = timed(lambda: qift.qift_diag_bucket_stats(W, codes, s, lloyd), 10)
    n, ratios = 100_000, [0.005 * i for i in range(1, 200)]
    x = torch.randn(n, device="cuda")
    ws = torch.empty(qift.qift_diag_ratio_scan_workspace_bytes(n, len(ratios)), dtype=torch.uint8, device="cuda")
    ms_r = timed(lambda: qift.qift_diag_ratio_scan(x, ratios, workspace=ws), 10)
    _, nmse = qift.qift_diag_ratio_scan(x, ratios, workspace=ws)
    gbs = N * K * 5 / (ms_b * 1e-3) / 1e9
    return {"workload": "Sec. 4.5 diagnostics on synthetic Gaussian weights",
            "bucket_stats": {"shape": [N, K], "us": round(ms_b * 1e3, 1), "value": round(gbs, 1), "unit": "GB/s",
                             "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 3)},
            "grid_quantize_mse_sweep": {"shape": [N, K], "grid": "Lloyd-Max", "us": round(ms_q * 1e3, 1),
                                        "candidate_evaluations_per_s": round(N * K * 80 / (ms_q * 1e-3), 0)},
            "ratio_scan": {"samples": n, "ratios": len(ratios), "us": round(ms_r * 1e3, 1),
                           "best_ratio": round(ratios[int(nmse.argmin())], 3), "best_nmse": round(float(nmse.min()), 6)}}


def int8_library_point(torch, M, shapes, device):
    """cuBLASLt int8 GEMM (torch._int_mm) on the same shapes: a library reference for the tensor-core rate."""
    try:
        ops, ms_total = 0.0, 0.0
        for (_, N, K) in shapes:
            a = torch.randint(-8, 8, (M, K), dtype=torch.int8, device=device)
            b = torch.randint(-3, 4, (N, K), dtype=torch.int8, device=device).t()
            for _ in range(3):
                torch._int_mm(a, b)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            ms_total += e0.elapsed_time(e1) / 10
            ops += 2.0 * M * N * K
        return {"api": "torch._int_mm (int8 x int8 -> int32, no scales, no decode)", "ms_per_layer": round(ms_total, 4),
                "tops": round(ops / (ms_total * 1e-3) / 1e12, 1)}
    except Exception as e:  # noqa: BLE001
        return {"api": "torch._int_mm", "unavailable": str(e)[:120]}


def run_prefill(torch, qift, L, device, gen, pk):
    """Config 4: LLaMA-3.1-8B shapes, M = 2048 tokens, bf16 in, bf16 out, MNZ."""
    M = 2048
    mods = build_stack(torch, qift, synth.LLAMA31_8B, 1, M, lambda l: qift.MNZ, 4000, torch.bfloat16, torch.bfloat16, device, gen)
    kmax = max(m.K for m in mods)
    q_a = torch.empty((M, kmax), dtype=torch.int8, device=device)
    s_a = torch.empty((M,), dtype=torch.float32, device=device)
    ws_bytes = max(qift.qift_workspace_bytes(M, m.N, m.K, m.levels) for m in mods)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
    vp = ctypes.c_void_p
    st = vp(torch.cuda.current_stream().cuda_stream)

    def layer(with_quant=True):
        for m in mods:
            if with_quant:
                rc = L.qift_quantize_act(vp(m.x.data_ptr()), qift.BF16, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st)
                assert rc == 0, rc
            rc = L.qift_w2a4_linear(vp(m.packed.data_ptr()), vp(m.s_n.data_ptr()), m.levels, vp(q_a.data_ptr()), vp(s_a.data_ptr()),
                                    M, m.N, m.K, vp(m.y.data_ptr()), qift.BF16, None, vp(ws.data_ptr()), ws_bytes, st)
            assert rc == 0, rc

    # resident decoded weights: one int8 level per weight kept beside the packed codes (decoded once, untimed)
    for m in mods:
        m.levels_i8 = qift.qift_expand_weights(m.packed, m.N, m.K, m.levels)

    def layer_resident(with_quant=True):
        for m in mods:
            if with_quant:
                rc = L.qift_quantize_act(vp(m.x.data_ptr()), qift.BF16, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st)
                assert rc == 0, rc
            rc = L.qift_expanded_linear(vp(m.levels_i8.data_ptr()), vp(m.s_n.data_ptr()), vp(q_a.data_ptr()), vp(s_a.data_ptr()),
                                        M, m.N, m.K, vp(m.y.data_ptr()), qift.BF16, None, st)
            assert rc == 0, rc

    def layer_resident_shared(_=True):
        # a transformer layer quantizes four inputs, not seven: q / k / v share one, gate / up share one
        for i, m in enumerate(mods):
            if m.name in ("q", "o", "gate", "down"):
                rc = L.qift_quantize_act(vp(m.x.data_ptr()), qift.BF16, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st)
                assert rc == 0, rc
            rc = L.qift_expanded_linear(vp(m.levels_i8.data_ptr()), vp(m.s_n.data_ptr()), vp(q_a.data_ptr()), vp(s_a.data_ptr()),
                                        M, m.N, m.K, vp(m.y.data_ptr()), qift.BF16, None, st)
            assert rc == 0, rc

    # the layer as it is usually deployed: q/k/v stored as one 6144 x 4096 matrix, gate/up as one 28672 x 4096 matrix
    # (same output channels, same ops), four quantized activations, resident decoded weights
    fused_shapes = [("qkv", 4096 + 1024 + 1024, 4096), ("o", 4096, 4096), ("gate_up", 2 * 14336, 4096), ("down", 4096, 14336)]
    fmods = build_stack(torch, qift, fused_shapes, 1, M, lambda l: qift.MNZ, 4100, torch.bfloat16, torch.bfloat16, device, gen)
    for m in fmods:
        m.levels_i8 = qift.qift_expand_weights(m.packed, m.N, m.K, m.levels)

    def layer_fused(_=True):
        for m in fmods:
            rc = L.qift_quantize_act(vp(m.x.data_ptr()), qift.BF16, M, m.K, m.B, CLIP, vp(q_a.data_ptr()), vp(s_a.data_ptr()), st)
            assert rc == 0, rc
            rc = L.qift_expanded_linear(vp(m.levels_i8.data_ptr()), vp(m.s_n.data_ptr()), vp(q_a.data_ptr()), vp(s_a.data_ptr()),
                                        M, m.N, m.K, vp(m.y.data_ptr()), qift.BF16, None, st)
            assert rc == 0, rc

    res = {}
    for key, fn, wq in (("layer_with_act_quant", layer, True), ("product_only", layer, False),
                        ("resident_fused_qkv_gateup", layer_fused, True),
                        ("resident_with_act_quant", layer_resident, True), ("resident_product_only", layer_resident, False),
                        ("resident_shared_act_quant", layer_resident_shared, True)):
        for _ in range(3):
            fn(wq)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        iters = 10
        e0.record()
        for _ in range(iters):
            fn(wq)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        ops = sum(2.0 * M * m.N * m.K for m in mods)
        res[key] = {"ms_per_layer": round(ms, 4), "tops": round(ops / (ms * 1e-3) / 1e12, 1)}
    res["resident_note"] = ("resident_*: the same layer through qift_expanded_linear on int8 levels decoded once "
                            "(4x the packed size, kept beside the packed codes); product_only decodes on every call; "
                            "resident_shared_act_quant quantizes the four distinct inputs of a layer (q/k/v and gate/up share "
                            "theirs) instead of one per module; resident_fused_qkv_gateup stores q/k/v and gate/up as "
                            "one matrix each (4 products + 4 quantizations per layer, same ops)")
    tops = res["product_only"]["tops"]
    gemm_tops = res["resident_product_only"]["tops"]      # the GEMM kernel alone (no decoding pass in the timed region)
    int8_peak = 2.0 * pk["bf16_tflops"]    # dense int8 is nominally 2x bf16; scaled from the measured bf16 burst
    res.update({"workload": "config 4: LLaMA-3.1-8B shapes, M=2048, 7 modules, MNZ, bf16 out", "unit": "TOPS",
                "pct_of_nominal_4500": round(100 * tops / 4500.0, 2),
                "resident_pct_of_nominal_4500": round(100 * gemm_tops / 4500.0, 2),
                "roofline": {"bound": "tensor", "kernel": "gemm_i8_pair_kernel", "achieved": gemm_tops,
                             "peak": int8_peak, "unit": "TOP/s", "frac": round(gemm_tops / int8_peak, 4),
                             "peak_source": f"2 x {pk['source']} bf16 burst",
                             "with_decoding_pass": {"kernels": "expand_levels_kernel + gemm_i8_pair_kernel", "achieved": tops,
                                                    "frac": round(tops / int8_peak, 4)}},
                "tokens_per_s": round(M / (res["layer_with_act_quant"]["ms_per_layer"] * 1e-3), 1),
                "resident_tokens_per_s": round(M / (res["resident_with_act_quant"]["ms_per_layer"] * 1e-3), 1),
                "fused_layer_tokens_per_s": round(M / (res["resident_fused_qkv_gateup"]["ms_per_layer"] * 1e-3), 1)})
    res["library_int8"] = int8_library_point(torch, M, synth.LLAMA31_8B, device)
    return res


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (baseline / reference arm)
# ------------------------------------------------------------------------------------------------
def oracle_layer_inputs():
    import oracle
    mods = []
    for i, (name, N, K) in enumerate(synth.LLAMA2_7B):
        rng = np.random.default_rng(2000 + i)
        codes = rng.integers(0, 4, (N, K), dtype=np.uint8)      # timing only: any codes cost the same
        s_n = np.full((N,), 0.01, dtype=np.float32)
        x, _ = synth.activations(synth.config_seed(2, i, 1), 1, K, max(1, round(0.01 * K)))
        mods.append((name, N, K, codes, s_n, x))
    return oracle, mods


def oracle_layer_once(oracle, mods):
    for (_, N, K, codes, s_n, x) in mods:
        q_a, s_a = oracle.quantize_act(x, synth.had_block_for(K), CLIP)
        oracle.linear(codes, oracle.MNZ, s_n, q_a, s_a)


def layer_bytes():
    return sum(product_bytes(1, N, K) + quant_bytes(1, K) for _, N, K in synth.LLAMA2_7B)


def cpu_baseline(budget_s=12.0):
    oracle, mods = oracle_layer_inputs()
    oracle_layer_once(oracle, mods)
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle_layer_once(oracle, mods)
        reps += 1
        if time.perf_counter() - t0 > budget_s or reps >= N_LAYERS:
            break
    dt = time.perf_counter() - t0
    return {"value": round(reps * layer_bytes() / dt / 1e9, 4), "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"{reps} of 32 layers (7 modules each, M=1) of the same workload, single thread, {dt:.1f} s",
            "host": f"{os.cpu_count()} logical cores"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    oracle, mods = oracle_layer_inputs()
    for _ in range(max(1, min(args.warmup, 2))):
        oracle_layer_once(oracle, mods)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_layer_once(oracle, mods)
    dt = time.perf_counter() - t0
    # one reference "step" is a bounded sample: 1 of the 32 layers; scale to the full step
    step_s = dt / steps * N_LAYERS
    value = N_LAYERS * layer_bytes() / step_s / 1e9
    sample = f"each step = 1 of 32 layers (7 modules, M=1), {steps} steps, single thread; ms_per_step scaled x32"
    print(json.dumps({
        "impl": "reference", "metric": "w2a4_decode_hbm_gbs", "value": round(value, 4), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": args.warmup,
        "ms_per_step": round(step_s * 1e3, 2), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": "config 2: LLaMA-2-7B-shaped decode, M=1, 7 linear shapes x 32 layers, MNZ; CPU oracle"},
        "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=N_LAYERS, help="layers of distinct weights per step (32 = the full workload)")
    ap.add_argument("--no-prefill", action="store_true", help="skip the M=2048 prefill measurement")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
