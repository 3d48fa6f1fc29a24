#!/usr/bin/env python
"""Sweep report (the outlier configuration and the N sweep of the benchmark definition); prints one JSON document.

    python bench_sweep.py [--quick]

* attention: N in {4096, 16384, 32768, 65536}, H=40, d=128, variants {bf16 (this repo's kernel),
  OCP direct, UOS direct, UOS+PNQ, UOS+PNQ+Hadamard}: kernel-only ms / TFLOP/s, whole-step ms, and the
  relative L2 error against float64 dense softmax attention on sampled rows (evaluated here with plain
  torch float64 operations on the GPU: a measurement aid, independent of both the kernels and the test oracle);
* outlier config (H=24, N=8192): the same quality comparison;
* row-sum diagnostic (Section 5.3): mean row sum of the quantized materialized probabilities and its split
  by quantization outcome, OCP / UOS / UOS+Hadamard, on three synthetic recipes at N=4096;
* short key/value sequences (cross-attention shapes): H=37, Nq=16384, 1 .. 96 KV tiles of 128 keys, attention launch
  only on pre-quantized operands: time and TFLOP/s (up to 48 tiles the launch uses the item-walking variant);
* Q_max study (paper Section 5.4.1 and its table of per-block optima): the ceiling-family boundary swept from 6.00 to
  8.00 in steps of 0.05 with mxattn_quantize_mxfp4_qmax on synthetic Q, K, V of 40 heads per recipe (the heads stand in
  for the paper's 40 attention blocks): tensor MSE per point, and the histogram of the per-head optimum;
* quantize: 2^20 .. 2^29 bf16 elements, axis 1 and axis 0, OCP and UOS: GB/s and fraction of the
  measured HBM copy rate.

The contract benchmark is bench.py; this script only adds the sweep tables.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402
from bench import QUANT_BYTES_PER_ELEM, load_peaks  # noqa: E402


SOFTMAX_PHASES = ["wait_scores", "load_scores", "maxima", "pair_exchange", "wait_prev_output_product", "block_exponents",
                  "exponentials_pack", "hand_over", "epilogue_per_item"]


def cycle_profile(mx, torch, cfg, dev):
    """Per-role cycle budget of the UOS + PNQ attention kernel (mxattn_forward_cycle_profile, the kernel compiled with
    cycle counters): mean SM cycles per key tile in each phase, per role, next to the time of the kernel without counters."""
    B, H, Nq, Nkv, d = cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d
    q, k, v = si.make_all(cfg)
    dq, dk, dv = dev(q), dev(k), dev(v)
    out = torch.empty((B, H, Nq, d), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
    flags = mx.FLAG_UOS | mx.FLAG_PNQ
    prof = torch.zeros(mx.forward_cycle_profile_bytes(B, H, Nq, Nkv, d) // 8, dtype=torch.int64, device="cuda")

    def timed(fn, n=5):
        fn(); torch.cuda.synchronize()
        ts = []
        for _ in range(n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return sorted(ts)[n // 2]

    ms_plain = timed(lambda: mx.forward_ws(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, flags, ws))
    ref = out.clone()
    ms_prof = timed(lambda: mx.forward_cycle_profile(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, flags, ws, prof))
    assert mx.device_status(ws) == 0 and torch.equal(out, ref)
    p = prof.view(-1, 18, 16).cpu().numpy().astype(np.float64)
    p = p[p[:, 17, 9] > 0]                                    # CTAs that ran (one per SM in the item-walking variant)
    tiles = p[:, 17, 9][:, None]
    kv_tiles = -(-Nkv // 128)
    sm = p[:, :16, :]
    per_tile = sm[:, :, :8] / np.maximum(sm[:, :, 9:10], 1)   # [cta, warp, phase]
    rep = {"workload": cfg.name, "H": H, "Nq": Nq, "Nkv": Nkv, "kv_tiles": kv_tiles, "ctas": int(p.shape[0]),
           "ms_without_counters": ms_plain, "ms_with_counters": ms_prof,
           "softmax_cycles_per_tile": {SOFTMAX_PHASES[i]: float(per_tile[:, :, i].mean()) for i in range(8)},
           "softmax_epilogue_cycles_per_item": float((sm[:, :, 8] / np.maximum(sm[:, :, 9] / kv_tiles, 1)).mean()),
           "issuer_cycles_per_tile": {"loop_total": float((p[:, 17, 8:9] / tiles).mean()),
                                      "wait_p_hat_tile0": float((p[:, 17, 0:1] / tiles).mean()), "wait_p_hat_tile1": float((p[:, 17, 2:3] / tiles).mean()),
                                      "wait_q": float((p[:, 17, 5:6] / tiles).mean()), "wait_kv": float((p[:, 17, 6:7] / tiles).mean()),
                                      "wait_score_buffer": float((p[:, 17, 7:8] / tiles).mean())},
           "producer_cycles_per_tile": {"loop_total": float((p[:, 16, 8:9] / tiles).mean()), "wait_free_stage": float((p[:, 16, 3:4] / tiles).mean()),
                                        "wait_free_q_buffer": float((p[:, 16, 5:6] / tiles).mean())}}
    rep["softmax_cycles_per_tile"]["sum"] = float(per_tile.sum(axis=2).mean())
    for g in (0, 1):            # the two softmax groups (query tile 0: warps 0-7, query tile 1: warps 8-15) separately
        pg = per_tile[:, 8 * g:8 * g + 8, :]
        rep[f"softmax_group{g}_cycles_per_tile"] = {SOFTMAX_PHASES[i]: float(pg[:, :, i].mean()) for i in range(8)}
    rep["issuer_cycles_per_tile"]["issuing"] = rep["issuer_cycles_per_tile"]["loop_total"] - sum(
        v for k_, v in rep["issuer_cycles_per_tile"].items() if k_.startswith("wait"))
    return rep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="smallest sizes only")
    ap.add_argument("--cycle-profile", default=None, metavar="WORKLOAD",
                    help="only this: per-role cycle profile of the attention kernel on the named workload (e.g. sweep16384, wan22, wan22_cross)")
    args = ap.parse_args()
    import torch
    import paper_2607_24377_b200 as mx
    peaks = load_peaks()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)
    f64 = lambda a: si.bf16_bits_to_f32(a).astype(np.float64)

    def timed(fn, n=3):
        fn(); torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            fn()
        b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def attention_report(cfg, heads_for_quality=(0, 1), rows_per_head=32):
        B, H, Nq, Nkv, d = cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d
        q, k, v = si.make_all(cfg)
        dq, dk, dv = dev(q), dev(k), dev(v)
        out = torch.empty((B, H, Nq, d), dtype=torch.float32, device="cuda")
        ws = torch.empty(mx.forward_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
        wsb = torch.empty(mx.forward_bf16_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
        rows = {h: np.sort(np.random.default_rng([5, h]).choice(Nq, rows_per_head, replace=False)) for h in heads_for_quality}
        def dense_rows(h):       # float64 softmax(Q K^T * scale) V for the sampled rows of head h, plain torch ops
            q64 = torch.from_numpy(f64(q[0, h][rows[h]])).cuda()
            k64 = torch.from_numpy(f64(k[0, h])).cuda()
            v64 = torch.from_numpy(f64(v[0, h])).cuda()
            sc = (q64 @ k64.T) * float(np.float32(cfg.softmax_scale))
            return (torch.softmax(sc, dim=1) @ v64).cpu().numpy()
        dense = {h: dense_rows(h) for h in heads_for_quality}

        def quality():
            num = den = 0.0
            for h in heads_for_quality:
                got = out[0, h][torch.from_numpy(rows[h]).cuda()].double().cpu().numpy()
                num += float(((got - dense[h]) ** 2).sum()); den += float((dense[h] ** 2).sum())
            return (num / den) ** 0.5

        rep = {"B": B, "H": H, "N": Nq, "flops": cfg.flops, "variants": {}}
        F32 = mx.FLAG_OUT_FP32
        for name, fl in (("ocp_direct", 0), ("uos_direct", mx.FLAG_UOS), ("uos_pnq", mx.FLAG_UOS | mx.FLAG_PNQ),
                         ("uos_pnq_hadamard", mx.FLAG_UOS | mx.FLAG_PNQ | mx.FLAG_HADAMARD)):
            ms = timed(lambda: mx.forward_ws(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, fl | F32, ws))
            assert mx.device_status(ws) == 0
            rep["variants"][name] = {"step_ms": ms, "step_tflops": cfg.flops / ms / 1e9, "rel_l2_vs_float64_dense": quality()}
        wsn = torch.empty(mx.forward_nvfp4_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
        for name, fl in (("nvfp4_direct", 0), ("nvfp4_pnq", mx.FLAG_PNQ)):      # the paper's comparison format, same kernel design
            ms = timed(lambda: mx.forward_nvfp4(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, fl | F32, wsn))
            assert mx.device_status(wsn) == 0
            rep["variants"][name] = {"step_ms": ms, "step_tflops": cfg.flops / ms / 1e9, "rel_l2_vs_float64_dense": quality()}
        del wsn
        ms = timed(lambda: mx.forward_bf16(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, F32, wsb))
        assert mx.device_status(wsb) == 0
        rep["variants"]["bf16_same_kernel"] = {"step_ms": ms, "step_tflops": cfg.flops / ms / 1e9, "rel_l2_vs_float64_dense": quality()}
        return rep

    if args.cycle_profile:
        print(json.dumps(cycle_profile(mx, torch, si.CONFIGS[args.cycle_profile], dev)))
        return

    doc = {"peaks": peaks, "attention_sweep": [], "quantize_sweep": []}
    sizes = (4096,) if args.quick else (4096, 16384, 32768, 65536)
    for n in sizes:
        doc["attention_sweep"].append(attention_report(si.CONFIGS[f"sweep{n}"]))
        torch.cuda.empty_cache()
    doc["outlier_config"] = attention_report(si.CONFIGS["outlier"], heads_for_quality=(0, 7, 15, 23), rows_per_head=16)
    torch.cuda.empty_cache()

    # row-sum diagnostic of Section 5.3 on synthetic rows (means over all rows of the config)
    doc["rowsum_diagnostic"] = []
    for name, cfg in (("iid N=4096", si.custom_config("iid4096", 1, 8, 4096, 4096, 11)),
                      ("wan recipe N=4096", si.custom_config("wan4096", 1, 8, 4096, 4096, 12, "wan")),
                      ("outlier recipe N=4096", si.CONFIGS["sweep4096"])):
        q, k, _ = si.make_all(cfg)
        dq, dk = dev(q), dev(k)
        out6 = torch.empty((cfg.B, cfg.H, cfg.Nq, 6), dtype=torch.float32, device="cuda")
        ws = torch.empty(mx.forward_workspace_bytes(cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d), dtype=torch.uint8, device="cuda")
        for label, fl in (("ocp", 0), ("uos", mx.FLAG_UOS), ("uos_hadamard", mx.FLAG_UOS | mx.FLAG_HADAMARD)):
            ms = timed(lambda: mx.rowsum_diagnostic(dq, dk, out6, cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d, cfg.softmax_scale, fl, ws))
            assert mx.device_status(ws) == 0
            o = out6.double().cpu().numpy().reshape(-1, 6)
            doc["rowsum_diagnostic"].append({
                "data": name, "rule": label, "ms": ms, "mean_row_sum": float(o[:, 0].mean()),
                "zeroing": float(o[:, 1].mean()), "saturation": float(o[:, 2].mean()), "downward": float(o[:, 3].mean()),
                "upward": float(o[:, 4].mean()), "mean_entropy": float(o[:, 5].mean()),
                "frac_rows_under_normalized": float((o[:, 0] < 1.0).mean())})
        torch.cuda.empty_cache()

    # short key/value sequences: the attention launch alone (operands quantized once, outside the timed region)
    doc["short_kv"] = []
    H, Nq = 37, 16384
    xq = torch.randn((1, H, Nq, 128), device="cuda").to(torch.bfloat16)
    out = torch.empty((1, H, Nq, 128), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    for tiles in ((1, 4) if args.quick else (1, 2, 4, 8, 16, 32, 48, 64, 96)):
        Nkv = 128 * tiles
        xk = torch.randn((1, H, Nkv, 128), device="cuda").to(torch.bfloat16)
        xv = torch.randn((1, H, Nkv, 128), device="cuda").to(torch.bfloat16)
        bufs = []
        for x, axis, n in ((xq, 1, Nq), (xk, 1, Nkv), (xv, 0, Nkv)):
            nt = -(-n // 128)
            c = torch.empty((H, nt, 8192), dtype=torch.uint8, device="cuda")
            sc = torch.empty((H, nt, 512), dtype=torch.uint8, device="cuda")
            mx.quantize_mxfp4_batched(x, c, sc, H, n, 128, axis, mx.MODE_UOS, mx.LAYOUT_TILE)
            bufs += [c, sc]
        ms = timed(lambda: mx.forward_prequantized(*bufs, out, 1, H, Nq, Nkv, 128, 128 ** -0.5,
                                                   mx.FLAG_UOS | mx.FLAG_PNQ, status), n=10)
        assert int(status[0]) == 0
        doc["short_kv"].append({"H": H, "Nq": Nq, "kv_tiles": tiles, "attn_us": ms * 1e3,
                                "tflops": 4.0 * H * Nq * Nkv * 128 / ms / 1e9})
    del xq, out
    torch.cuda.empty_cache()

    # Q_max study: sweep of the ceiling-family boundary (Eq. 7) on synthetic tensors; 40 heads per recipe stand in for the
    # paper's 40 attention blocks.  Dequantization and the MSE are plain torch operations (a measurement aid).
    doc["qmax_study"] = []
    lut = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6], dtype=torch.float32, device="cuda")
    points = [round(6.0 + 0.05 * i, 2) for i in range(41)]
    Hq, Nq_ = (8, 1024) if args.quick else (40, 8192)
    for recipe, seed in (("iid", 21), ("outlier", 22), ("wan", 23), ("hunyuan", 24)):
        cfg = si.custom_config("qmax_" + recipe, 1, Hq, Nq_, Nq_, seed, recipe)
        q, k, v = si.make_all(cfg)
        for tname, bits, axis in (("Q", q, 1), ("K", k, 1), ("V", v, 0)):
            x = dev(bits)[0]                                            # [H, N, 128] bf16
            xf = x.float()
            codes = torch.empty((Hq, Nq_, 64) if axis == 1 else (Hq, 128, Nq_ // 2), dtype=torch.uint8, device="cuda")
            scales = torch.empty((Hq, Nq_, 4) if axis == 1 else (Hq, 128, Nq_ // 32), dtype=torch.uint8, device="cuda")
            mse = np.empty((len(points), Hq))
            for i, qm in enumerate(points):
                mx.quantize_mxfp4_qmax(x, codes, scales, Hq, Nq_, 128, axis, qm, mx.LAYOUT_CANONICAL)
                nib = torch.stack([codes & 15, codes >> 4], dim=-1).flatten(-2)              # [..., inner]
                val = lut[nib.long()] * torch.exp2(scales.float() - 127.0).repeat_interleave(32, dim=-1)
                if axis == 0:
                    val = val.transpose(1, 2)                                                # back to [H, N, 128]
                mse[i] = ((val - xf) ** 2).mean(dim=(1, 2)).double().cpu().numpy()
            best = np.array(points)[mse.argmin(axis=0)]                                      # per-head optimum
            curve = mse.mean(axis=1)
            doc["qmax_study"].append({
                "recipe": recipe, "tensor": tname, "heads": Hq, "tokens": Nq_,
                "argmin_of_mean_mse": points[int(curve.argmin())],
                "mse_at_6.00": float(curve[0]), "mse_at_7.00": float(curve[points.index(7.0)]),
                "mse_at_7.25": float(curve[points.index(7.25)]), "mse_at_8.00": float(curve[-1]),
                "pct_heads_optimum_le_7.15": float((best <= 7.151).mean() * 100), "pct_heads_optimum_7.20": float((np.abs(best - 7.20) < 1e-6).mean() * 100),
                "pct_heads_optimum_7.25": float((np.abs(best - 7.25) < 1e-6).mean() * 100), "pct_heads_optimum_ge_7.30": float((best >= 7.299).mean() * 100),
                "mean_mse_curve": [float(c) for c in curve]})
        torch.cuda.empty_cache()

    exps = (20, 24) if args.quick else range(20, 30)
    for e in exps:
        n = 1 << e
        rows = n // 128
        x = torch.randn((rows, 128), device="cuda").to(torch.bfloat16)
        for axis in (1, 0):
            batch = max(1, rows // 8192) if axis == 0 else 1
            r = rows // batch
            rp = -(-r // 128) * 128
            codes = torch.empty(batch * max(r, rp) * 64 if axis == 1 else batch * 128 * rp // 2, dtype=torch.uint8, device="cuda")
            scales = torch.empty(batch * max(r, rp) * 4, dtype=torch.uint8, device="cuda")
            for mode, mname in ((mx.MODE_OCP, "ocp"), (mx.MODE_UOS, "uos")):
                ms = timed(lambda: mx.quantize_mxfp4_batched(x, codes, scales, batch, r, 128, axis, mode, mx.LAYOUT_CANONICAL), n=10)
                gbs = QUANT_BYTES_PER_ELEM * n / ms / 1e6
                doc["quantize_sweep"].append({"elements": n, "axis": axis, "mode": mname, "ms": ms, "GBps": gbs,
                                              "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]})
        # NVFP4 (the comparison format): tensor maximum + quantizer, 2 + 2 + 0.5 + 1/16 bytes per element
        for axis in (1, 0):
            batch = max(1, rows // 8192)
            r = rows // batch
            rp = -(-r // 128) * 128
            codes = torch.empty(batch * max(r, rp) * 64, dtype=torch.uint8, device="cuda")
            scales = torch.empty(batch * max(r, rp) * 8, dtype=torch.uint8, device="cuda")
            amax = torch.empty(batch, dtype=torch.float32, device="cuda"); ts = torch.empty(batch, dtype=torch.float32, device="cuda")
            def nv():
                mx.tensor_amax(x, amax, batch, r, 128)
                mx.quantize_nvfp4(x, codes, scales, amax, ts, batch, r, 128, axis, mx.LAYOUT_CANONICAL)
            ms = timed(nv, n=10)
            gbs = (4.0 + 0.5 + 1.0 / 16.0) * n / ms / 1e6
            doc["quantize_sweep"].append({"elements": n, "axis": axis, "mode": "nvfp4 (tensor maximum + quantizer)", "ms": ms, "GBps": gbs,
                                          "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]})
        del x
    print(json.dumps(doc))


if __name__ == "__main__":
    main()
