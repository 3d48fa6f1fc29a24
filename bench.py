#!/usr/bin/env python
"""Benchmark of the MXAttention hot path on B200: one "step" = one full pass of Algorithm 2
lines 3-19 (quantize Q, K, V with UOS; fused PNQ attention forward) over one synthetic batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload wan22] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is whole-job TFLOP/s (4*B*H*Nq*Nkv*d per batch) with the
bf16 inputs already resident in HBM; `e2e` is the same metric through the host-buffer entry point
(pinned host tensors in, result out, copies inside the timed region).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "uos_pnq_mxfp4_attention_forward_tflops"
UNIT = "TFLOP/s"
NOMINAL_FP4_TFLOPS = 9000.0      # dense FP4, nominal
FP4_OVER_BF16 = 4.0              # nominal ratio of dense FP4 to dense bf16 tensor throughput
QUANT_BYTES_PER_ELEM = 2.0 + 0.5 + 1.0 / 32.0
# DRAM bytes of one attention launch, from the ncu capture of the same kernel on sweep16384
# (259.4 MB, profiles/attention_kernel_sweep16384.txt) scaled by tokens x heads (traffic follows the
# operand bytes, not the flops; valid for the self-attention workloads, Nq = Nkv).
ATTN_TRAFFIC_PER_TOKEN_HEAD = 259.4e6 / (16384 * 40)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        """gpu_id: what nvidia-smi's -i takes.  The GPU's UUID, not the CUDA ordinal: nvidia-smi numbers the
        machine's GPUs physically and ignores CUDA_VISIBLE_DEVICES, so an ordinal can name another job's GPU."""
        super().__init__(daemon=True)
        self.index, self.samples, self._stop_evt, self.proc = gpu_id, [], threading.Event(), None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                if self._stop_evt.is_set():
                    break
                self.samples.append([x.strip() for x in line.split(",")])
        except Exception:
            pass

    def stop(self):
        self._stop_evt.set()
        if self.proc is not None:
            self.proc.terminate()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0])); mx = max(mx, float(s[1]))
                for n, v in zip(names, s[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "gpu": self.index}
        # median over the samples taken under load (upper half)
        hot = sorted(sm)[len(sm) // 2:]
        return {"sm_mhz": float(np.median(hot)), "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm),
                "gpu": self.index}


def gpu_uuid(torch, local: int) -> str:
    u = str(torch.cuda.get_device_properties(local).uuid)
    return u if u.startswith("GPU-") else "GPU-" + u


# ----------------------------------------------------------------------------------------------
def oracle_sample(cfg, heads, rows_per_head, inputs=None, threads=None):
    """Times the CPU oracle (as it stands) on sampled query rows of `cfg`; returns (TFLOP/s-equivalent, seconds, desc).
    inputs: optional {head: (q, k, v)} generated beforehand (then input generation is outside the timed region).
    threads: limit of the BLAS thread pool the oracle's NumPy calls use (None: whatever the environment gives)."""
    from oracle import attention
    import contextlib
    limit = contextlib.nullcontext()
    if threads is not None:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=threads)
    f = lambda a: si.bf16_bits_to_f32(a).astype(np.float64)
    n_rows = 0
    with limit:
        t0 = time.perf_counter()
        for h in heads:
            q, k, v = inputs[h] if inputs is not None else si.make_head(cfg, 0, h)
            rng = np.random.default_rng([99, h])
            rows = np.sort(rng.choice(cfg.Nq, rows_per_head, replace=False))
            attention.forward_head(f(q), f(k), f(v), cfg.softmax_scale, True, True, rows=rows)
            n_rows += rows_per_head
        dt = time.perf_counter() - t0
    flops = 4.0 * n_rows * cfg.Nkv * cfg.d
    return flops / dt / 1e12, dt, f"{rows_per_head} random query rows x all {cfg.Nkv} keys in each of heads {list(heads)} " \
                                  f"(quantization of those heads' Q, K, V included" + \
                                  (")" if inputs is not None else ", input generation too)")


def probe_fp4_peak(mx, torch, gpu_id):
    """Measures what the FP4 tensor pipe of this GPU delivers with the library's own dense block-scaled FP4 GEMM
    (mxattn_probe_fp4_gemm, the same tcgen05.mma kind::mxf4.block_scale the attention kernel issues), with CUDA events
    and the SM clock sampled meanwhile.  Two figures: `streaming` -- an 8192^3 GEMM whose operands come from global
    memory --, and `resident` -- the same instruction stream with its operand ring loaded once (issue rate of the
    tensor pipe itself).  The roofline's denominator is the larger of the two."""
    M = N = K = 8192            # (in resident mode 2048 CTAs = 13.8 waves of 148: the partly filled last wave is part of the figure)
    kb = K // 128
    g = torch.Generator(device="cuda"); g.manual_seed(1)
    ops = []
    for rows in (M, N):
        codes = torch.randint(0, 256, (kb, rows // 128, 8192), dtype=torch.uint8, device="cuda", generator=g)
        scales = torch.randint(124, 131, (kb, rows // 128, 512), dtype=torch.uint8, device="cuda", generator=g)
        ops += [codes, scales]
    c = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    out = {"kernel": "fp4_gemm_probe_kernel (128 x tile_n tiles, kind::mxf4.block_scale, M = N = 8192)"}
    for name, k_steps, resident, tile_n in (("streaming", kb, False, 256), ("resident", 510, True, 256), ("resident_n128", 510, True, 128)):
        flops = 2.0 * M * N * 128 * k_steps
        for _ in range(3):
            mx.probe_fp4_gemm(*ops, c, M, N, K, k_steps, resident, False, status, tile_n)
        torch.cuda.synchronize()
        sampler = ClockSampler(gpu_id); sampler.start(); time.sleep(0.25)
        n = 12 if resident else 30
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        evs[0].record()
        for i in range(n):
            mx.probe_fp4_gemm(*ops, c, M, N, K, k_steps, resident, False, status, tile_n)
            evs[i + 1].record()
        torch.cuda.synchronize()
        time.sleep(0.15); sampler.stop()
        ms = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(n))
        clk = sampler.summary()
        out[name] = {"k_steps": k_steps, "tile_n": tile_n, "launches": n, "ms_best": ms[0], "ms_median": ms[n // 2],
                     "tflops_best": flops / (ms[0] * 1e-3) / 1e12, "tflops_median": flops / (ms[n // 2] * 1e-3) / 1e12,
                     "sm_mhz": clk["sm_mhz"], "reasons": clk["reasons"]}
    assert int(status[0].item()) == 0, "a bounded device-side wait expired in the FP4 GEMM probe"
    best = max(("streaming", "resident", "resident_n128"), key=lambda k: out[k]["tflops_median"])
    out["peak_tflops"] = out[best]["tflops_median"]
    out["peak_mode"] = best
    out["peak_sm_mhz"] = out[best]["sm_mhz"]
    return out


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    """--impl reference: the oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy  # noqa: F401  (BLAS threads are whatever the environment gives the oracle)
    heads = [0]
    rows = min(cfg.Nq, 256 if cfg.Nkv > 20000 else 512)     # a few seconds per step
    vals = []
    for i in range(args.warmup + args.steps):
        tf, dt, desc = oracle_sample(cfg, heads, rows)
        if i >= args.warmup:
            vals.append((tf, dt))
    tf = float(np.mean([v[0] for v in vals]))
    ms = float(np.mean([v[1] for v in vals]) * 1e3)
    line = {"metric": METRIC, "value": tf, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "Nq": cfg.Nq, "Nkv": cfg.Nkv, "d": cfg.d,
                       "step": "bounded sample of the workload: " + desc},
            "cpu_baseline": {"value": tf, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="wan22", choices=sorted(si.CONFIGS))
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-variants", action="store_true")
    ap.add_argument("--no-fp4-probe", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    cfg = si.CONFIGS[args.workload]

    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    import paper_2607_24377_b200 as mx

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()

    # ---- synthetic inputs (weak scaling: every rank owns one full batch, seeded by rank) ----
    rcfg = si.AttnConfig(cfg.name, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.seed + 1000 * rank, cfg.recipe)
    B, H, Nq, Nkv, d = cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d
    hq = torch.empty((B, H, Nq, d), dtype=torch.int16).pin_memory()
    hk = torch.empty((B, H, Nkv, d), dtype=torch.int16).pin_memory()
    hv = torch.empty((B, H, Nkv, d), dtype=torch.int16).pin_memory()
    for b in range(B):
        for h in range(H):
            q, k, v = si.make_head(rcfg, b, h)
            hq[b, h] = torch.from_numpy(q.view(np.int16)); hk[b, h] = torch.from_numpy(k.view(np.int16))
            hv[b, h] = torch.from_numpy(v.view(np.int16))
    dq, dk, dv = (t.cuda().view(torch.bfloat16) for t in (hq, hk, hv))
    out = torch.empty((B, H, Nq, d), dtype=torch.bfloat16, device="cuda")
    flags = mx.FLAG_UOS | mx.FLAG_PNQ
    ws_bytes = mx.forward_workspace_bytes(B, H, Nq, Nkv, d)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    bh, qt, kt = B * H, -(-Nq // 128), -(-Nkv // 128)
    # the same buffers mxattn_forward_ws carves from its workspace, held separately here so that
    # each of its four launches can be bracketed by CUDA events
    qc, qs = (torch.empty((bh, qt, n), dtype=torch.uint8, device="cuda") for n in (8192, 512))
    kc, ks = (torch.empty((bh, kt, n), dtype=torch.uint8, device="cuda") for n in (8192, 512))
    vc, vs = (torch.empty((bh, kt, n), dtype=torch.uint8, device="cuda") for n in (8192, 512))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    scale = cfg.softmax_scale

    def step(events=None, fl=flags):
        mode = mx.MODE_UOS if (fl & mx.FLAG_UOS) else mx.MODE_OCP
        ev = events or [None] * 5
        if ev[0]: ev[0].record()
        mx.quantize_mxfp4_batched(dq, qc, qs, bh, Nq, d, 1, mode, mx.LAYOUT_TILE)
        if ev[1]: ev[1].record()
        mx.quantize_mxfp4_batched(dk, kc, ks, bh, Nkv, d, 1, mode, mx.LAYOUT_TILE)
        if ev[2]: ev[2].record()
        mx.quantize_mxfp4_batched(dv, vc, vs, bh, Nkv, d, 0, mode, mx.LAYOUT_TILE)
        if ev[3]: ev[3].record()
        mx.forward_prequantized(qc, qs, kc, ks, vc, vs, out, B, H, Nq, Nkv, d, scale, fl, status)
        if ev[4]: ev[4].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    gpu_id = gpu_uuid(torch, local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    barrier()
    t_start = torch.cuda.Event(enable_timing=True); t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        step(evs[i])
    t_stop.record()
    barrier()
    if rank == 0:
        sampler.stop()
    assert int(status[0].item()) == 0, "a bounded device-side wait expired"
    from paper_2607_24377_b200 import sharding
    flops = cfg.flops
    value, ms_per_step = sharding.aggregate_throughput(flops, t_start.elapsed_time(t_stop) / args.steps, world, "cuda")
    value /= 1e12

    kern_ms = [float(np.mean([evs[i][a].elapsed_time(evs[i][a + 1]) for i in range(args.steps)])) for a in range(4)]
    attn_ms = kern_ms[3]
    attn_tflops = flops / (attn_ms * 1e-3) / 1e12
    # best and median of the attention launch over at least ten launches (the timed steps plus extra launches)
    attn_all = [evs[i][3].elapsed_time(evs[i][4]) for i in range(args.steps)]
    for _ in range(max(0, 10 - args.steps)):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        mx.forward_prequantized(qc, qs, kc, ks, vc, vs, out, B, H, Nq, Nkv, d, scale, flags, status)
        b.record(); torch.cuda.synchronize()
        attn_all.append(a.elapsed_time(b))
    attn_all.sort()
    attn_stats = {"launches": len(attn_all), "ms_best": attn_all[0], "ms_median": attn_all[len(attn_all) // 2],
                  "tflops_best": flops / (attn_all[0] * 1e-3) / 1e12,
                  "tflops_median": flops / (attn_all[len(attn_all) // 2] * 1e-3) / 1e12}
    q_elems = [bh * Nq * d, bh * Nkv * d, bh * Nkv * d]
    quant = {}
    for i, name in enumerate(("q_axis1", "k_axis1", "v_axis0")):
        gbps = QUANT_BYTES_PER_ELEM * q_elems[i] / (kern_ms[i] * 1e-3) / 1e9
        # two denominators: the copy rate measured on this machine (a plain copy, so a good kernel can read slightly
        # above 1) and the nominal 8 TB/s the metric names
        quant[name] = {"ms": kern_ms[i], "GBps": gbps, "frac_of_measured_copy_rate": gbps / peaks["hbm_gbs"],
                       "frac_of_nominal_8TBps": gbps / 8000.0}
    fp4 = None
    if not args.no_fp4_probe and rank == 0:
        fp4 = probe_fp4_peak(mx, torch, gpu_id)

    # ---- variants of the same kernel (kernel-only, a few launches each) ----
    variants = {}
    if not args.no_variants:
        for name, fl in (("ocp_direct", 0), ("uos_direct", mx.FLAG_UOS), ("ocp_pnq", mx.FLAG_PNQ), ("uos_pnq", flags)):
            step(fl=fl); torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n = 3
            a.record()
            for _ in range(n):
                mx.forward_prequantized(qc, qs, kc, ks, vc, vs, out, B, H, Nq, Nkv, d, scale, fl, status)
            b.record(); torch.cuda.synchronize()
            ms = a.elapsed_time(b) / n
            variants[name] = {"attn_ms": ms, "tflops": flops / (ms * 1e-3) / 1e12}
        variants["uos_pnq_over_ocp_direct_time"] = variants["uos_pnq"]["attn_ms"] / variants["ocp_direct"]["attn_ms"]
        # Algorithm 2 lines 1-2 fused into the Q/K quantize launches (the attention launch is unchanged)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        rot = mx.MODE_UOS | mx.MODE_HADAMARD
        mx.quantize_mxfp4_batched(dq, qc, qs, bh, Nq, d, 1, rot, mx.LAYOUT_TILE); torch.cuda.synchronize()
        a.record()
        for _ in range(3):
            mx.quantize_mxfp4_batched(dq, qc, qs, bh, Nq, d, 1, rot, mx.LAYOUT_TILE)
        b.record(); torch.cuda.synchronize()
        ms = a.elapsed_time(b) / 3
        gbps = QUANT_BYTES_PER_ELEM * q_elems[0] / (ms * 1e-3) / 1e9
        variants["quantize_q_with_hadamard"] = {"ms": ms, "GBps": gbps, "frac_of_measured_copy_rate": gbps / peaks["hbm_gbs"],
                                                "frac_of_nominal_8TBps": gbps / 8000.0}
        mx.quantize_mxfp4_batched(dq, qc, qs, bh, Nq, d, 1, mx.MODE_UOS, mx.LAYOUT_TILE)       # restore the unrotated Q-hat
        # bf16 variant of this repository's own kernel (no quantization; three re-tiling launches + attention)
        wsb = torch.empty(mx.forward_bf16_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
        mx.forward_bf16(dq, dk, dv, out, B, H, Nq, Nkv, d, scale, 0, wsb); torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(3):
            mx.forward_bf16(dq, dk, dv, out, B, H, Nq, Nkv, d, scale, 0, wsb)
        b.record(); torch.cuda.synchronize()
        assert mx.device_status(wsb) == 0
        ms = a.elapsed_time(b) / 3
        variants["bf16_same_kernel"] = {"step_ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                                        "note": "mxattn_forward_bf16: whole call (re-tiling of Q, K, V^T + fused attention)"}
        variants["uos_pnq_step_speedup_over_bf16_same_kernel"] = ms / ms_per_step
        del wsb
        # the paper's comparison format: the same kernel design on NVFP4 operands (whole call: three tensor maxima,
        # three quantize launches, attention)
        wsn = torch.empty(mx.forward_nvfp4_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
        for name, fl in (("nvfp4_direct", 0), ("nvfp4_pnq", mx.FLAG_PNQ)):
            mx.forward_nvfp4(dq, dk, dv, out, B, H, Nq, Nkv, d, scale, fl, wsn); torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(3):
                mx.forward_nvfp4(dq, dk, dv, out, B, H, Nq, Nkv, d, scale, fl, wsn)
            b.record(); torch.cuda.synchronize()
            assert mx.device_status(wsn) == 0
            ms = a.elapsed_time(b) / 3
            variants[name] = {"step_ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                              "note": "mxattn_forward_nvfp4: whole call (7 launches)"}
        del wsn
        # bf16 reference point: NOT a kernel of this repository -- PyTorch's fused SDPA (library flash /
        # cuDNN attention) on the same bf16 tensors.  (The repository's own bf16 variant is `bf16_same_kernel` above.)
        try:
            import torch.nn.functional as F
            ob = F.scaled_dot_product_attention(dq, dk, dv, scale=scale); del ob
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(2):
                ob = F.scaled_dot_product_attention(dq, dk, dv, scale=scale)
            b.record(); torch.cuda.synchronize(); del ob
            ms = a.elapsed_time(b) / 2
            variants["bf16_library_sdpa"] = {"attn_ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                                             "note": "torch.nn.functional.scaled_dot_product_attention, library kernel, context only"}
            variants["uos_pnq_speedup_over_bf16_library"] = ms / variants["uos_pnq"]["attn_ms"]
        except Exception as exc:  # pragma: no cover
            variants["bf16_library_sdpa"] = {"unavailable": str(exc)[:200]}

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not args.no_e2e:
        arena = torch.empty(mx.forward_host_arena_bytes(B, H, Nq, Nkv, d, flags), dtype=torch.uint8, device="cuda")
        ho = torch.empty((B, H, Nq, d), dtype=torch.int16).pin_memory()
        n_e2e = max(2, min(args.steps, 3))
        mx.forward_host(hq, hk, hv, ho, B, H, Nq, Nkv, d, scale, flags, arena)
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            mx.forward_host(hq, hk, hv, ho, B, H, Nq, Nkv, d, scale, flags, arena)   # synchronizes internally
        dt = (time.perf_counter() - t0) / n_e2e
        dt = sharding.max_over_ranks(dt, "cuda")
        e2e = {"value": world * flops / dt / 1e12, "unit": UNIT, "ms_per_step": dt * 1e3,
               "h2d_bytes_per_step": int(hq.numel() + hk.numel() + hv.numel()) * 2,
               "d2h_bytes_per_step": int(ho.numel()) * 2, "steps": n_e2e}
        del arena

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline:
        # the oracle as it stands on sampled rows spread over four heads, once on one thread and once on all host cores
        heads = sorted(set(int(h) for h in np.linspace(0, H - 1, 4)))
        rows = min(cfg.Nq, 384 if Nkv > 20000 else 1024)
        inputs = {h: si.make_head(cfg, 0, h) for h in heads}
        tf_all, dt_all, desc = oracle_sample(cfg, heads, rows, inputs=inputs)
        n_all = cpu_threads()
        tf_one, dt_one, _ = oracle_sample(cfg, heads, rows, inputs=inputs, threads=1)
        cpu_baseline = {"value": tf_all, "unit": UNIT, "cores": n_all, "kind": "oracle", "sample": desc, "seconds": dt_all,
                        "single_thread": {"value": tf_one, "unit": UNIT, "cores": 1, "seconds": dt_one},
                        "host_cpus": os.cpu_count(),
                        "extrapolated_full_workload_hours": cfg.flops / (tf_all * 1e12) / 3600.0}

    clocks = sampler.summary()
    mufu_ceiling = 16 * 512 * 148 * clocks["sm_mhz"] * 1e6 / 1e12 if clocks.get("sm_mhz") else None
    # Roofline of the dominant kernel.  Denominator: the dense FP4 rate measured just above with the library's own
    # block-scaled GEMM probe ("of measured"); without the probe, the measured sustained cuBLAS bf16 rate times
    # the nominal FP4 : bf16 ratio.  The two measurements run at different SM clocks (a saturated tensor pipe is
    # power-capped, this kernel is not), so the fraction is also given per clock: flops per SM cycle over flops per
    # SM cycle.  What binds this kernel is not the tensor pipe but the exponential unit (one ex2 per score, 16 per
    # clock and SM against 64 scores' worth of FP4 flops), hence "bound": "mufu" and the fraction of that ceiling.
    if fp4:
        fp4_peak = fp4["peak_tflops"]
        peak_note = (f"dense FP4 measured in this run: mxattn_probe_fp4_gemm, {fp4['peak_mode']} mode, median of "
                     f"{fp4[fp4['peak_mode']]['launches']} launches at {fp4['peak_sm_mhz']} MHz (of measured)")
        per_clock = None
        if clocks.get("sm_mhz") and fp4.get("peak_sm_mhz"):
            per_clock = (attn_tflops / clocks["sm_mhz"]) / (fp4_peak / fp4["peak_sm_mhz"])
    else:
        fp4_peak = peaks["bf16_tflops_sustained"] * FP4_OVER_BF16
        peak_note = (f"no FP4 probe in this run: {peaks['source']} sustained bf16 cuBLAS {peaks['bf16_tflops_sustained']} "
                     f"x nominal ratio 4 (of {peaks['source']})")
        per_clock = None
    roofline = {"bound": "mufu", "kernel": "attention_kernel<uos,pnq>", "achieved": attn_tflops,
                "peak": fp4_peak, "unit": "TFLOP/s", "frac": attn_tflops / fp4_peak,
                "frac_per_sm_clock": per_clock, "achieved_sm_mhz": clocks.get("sm_mhz"),
                "traffic": ATTN_TRAFFIC_PER_TOKEN_HEAD * Nkv * B * H if Nq == Nkv else None,
                "traffic_note": "ncu dram bytes of a sweep16384 launch scaled by tokens x heads",
                "peak_note": peak_note,
                "frac_of_nominal_9PF": attn_tflops / NOMINAL_FP4_TFLOPS, "launch_ms": attn_ms,
                # the softmax exponentials bind before the tensor pipe does: 16 ex2 per clock per SM,
                # one per (query, key) pair, 512 tensor flops per pair
                "mufu_ceiling_tflops": mufu_ceiling, "frac_of_mufu_ceiling": attn_tflops / mufu_ceiling if mufu_ceiling else None,
                "ncu_cross_check": "profiles/attention_kernel_sweep16384.txt: sm__pipe_tensor_cycles_active 21.2 %, XU pipe 83 %"}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp4 (E2M1 x E8M0, fp32 accumulate)", "data": "synthetic",
        "config": {"workload": cfg.name, "B": B, "H": H, "Nq": Nq, "Nkv": Nkv, "d": d, "flags": "uos|pnq",
                   "out": "bf16", "l2": "inputs (2.3 GB at wan22) exceed L2; no flush needed",
                   "sharding": "one full batch per GPU, no collective"},
        "clocks": clocks,
        "e2e": e2e, "gpu_launches": 4 * args.steps,
        "roofline": roofline,
        "fp4_peak_probe": fp4,
        "attention_launch": attn_stats,
        "cpu_baseline": cpu_baseline,
        "kernels_ms": {"quantize_q": kern_ms[0], "quantize_k": kern_ms[1], "quantize_v": kern_ms[2], "attention": attn_ms},
        "quantize": quant, "variants": variants,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
