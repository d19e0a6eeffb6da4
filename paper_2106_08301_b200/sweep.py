"""Timing sweep over the synthetic workloads (one JSON line per workload on stdout).

For each workload: mwu_project, mwu_pack and mwu_gemm (or mwu_conv_implicit) are timed with CUDA
events on the launching stream, L2 is flushed between repetitions (a 256 MB buffer is rewritten),
and the dense bf16 library routine (torch.matmul / conv2d on the decoded weights) is timed beside
them.  Roofline time = max(surviving-block FLOPs / tensor peak, algorithmic bytes / HBM peak).

  python -m paper_2106_08301_b200.sweep [--set main|blocks|projection|all] [--reps 10] [--m M] [--fused]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2106_08301_b200 import binding as B  # noqa: E402
from paper_2106_08301_b200 import inputs  # noqa: E402


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return d["hbm_gbs"], d["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


class Timer:
    def __init__(self):
        self.flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    def time(self, fn, reps, flush=True):
        out = []
        for _ in range(reps):
            if flush:
                self.flush.fill_(1)
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1))
        return statistics.median(out), min(out)


def packed_algorithmic_bytes(wl, ku, kp):
    n_u, n_d = ku - kp, wl.n_blocks - ku
    return (2 * kp + n_u * (32 + wl.block + 2) + n_d * (16 * wl.block + 2)) / 8.0


def run_workload(wl, timer, reps, m_override=None, fused=False):
    hbm, tf, src = peaks()
    ku = B.mwu_count_from_permille(wl.n_blocks, wl.unified_permille)
    kp = B.mwu_count_from_permille(wl.n_blocks, wl.pruned_permille)
    desc = B.make_desc(wl.rows, wl.cols, wl.block, ku, kp)
    W = wl.weights().cuda()
    bufs = B.ProjectionBuffers(desc, want_q=True)
    packed = torch.empty(B.mwu_packed_bytes(desc), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        bufs.project(W)
        bufs.pack(W, packed=packed)
    torch.cuda.synchronize()
    proj_ms, proj_best = timer.time(lambda: bufs.project(W), reps)
    pack_ms, _ = timer.time(lambda: bufs.pack(W, packed=packed), reps)
    Wd = bufs.Q.reshape(wl.rows, wl.cols).to(torch.bfloat16)
    res = {"workload": wl.name, "rows": wl.rows, "cols": wl.cols, "block": wl.block, "k_unify": ku,
           "k_prune": kp, "project_ms": proj_ms, "pack_ms": pack_ms,
           "projection_gbs_algorithmic": 8.0 * wl.rows * wl.cols / (proj_ms * 1e-3) / 1e9,
           "projection_frac_of_hbm": 8.0 * wl.rows * wl.cols / (proj_ms * 1e-3) / 1e9 / hbm,
           "peaks": src}
    if wl.conv is not None:
        n, c, h, w, kh, kw, stride, pad = wl.conv
        X = wl.activations().cuda()
        oh = (h + 2 * pad - kh) // stride + 1
        ow = (w + 2 * pad - kw) // stride + 1
        Y = torch.empty((n, wl.rows, oh, ow), dtype=torch.bfloat16, device="cuda")
        m = n * oh * ow

        def call():
            B.mwu_conv_implicit(desc, packed, X, n, c, h, w, kh, kw, stride, pad, Y, 0, bufs.dev_status)

        W4 = Wd.reshape(wl.rows, c, kh, kw)

        def lib():
            torch.nn.functional.conv2d(X, W4, stride=stride, padding=pad)
    else:
        m = m_override or wl.m
        X = wl.activations(m=m).cuda()
        Y = torch.empty((m, wl.rows), dtype=torch.bfloat16, device="cuda")
        ws_bytes = 0 if fused else B.mwu_gemm_workspace_bytes(desc, m)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
        res["gemm_path"] = "decode once" if ws_bytes else "fused decode"

        def call():
            B.mwu_gemm_ws(desc, packed, X, m, wl.cols, Y, wl.rows, 0, ws, bufs.dev_status)

        def lib():
            torch.matmul(X, Wd.T)
    for _ in range(3):
        call()
        lib()
    torch.cuda.synchronize()
    gemm_ms, gemm_best = timer.time(call, reps)
    lib_ms, _ = timer.time(lib, reps)
    flops = 2.0 * m * wl.block * (wl.n_blocks - kp)
    dense = 2.0 * m * wl.rows * wl.cols
    bytes_ = 2.0 * m * wl.cols + 2.0 * m * wl.rows + packed_algorithmic_bytes(wl, ku, kp)
    if wl.conv is not None:
        n, c, h, w = wl.conv[:4]
        bytes_ = 2.0 * n * c * h * w + 2.0 * m * wl.rows + packed_algorithmic_bytes(wl, ku, kp)
    roof_ms = max(flops / (tf * 1e12), bytes_ / (hbm * 1e9)) * 1e3
    res.update({"m": m, "gemm_ms": gemm_ms, "gemm_best_ms": gemm_best, "library_dense_bf16_ms": lib_ms,
                "effective_tflops": flops / (gemm_ms * 1e-3) / 1e12,
                "executed_dense_tflops": dense / (gemm_ms * 1e-3) / 1e12,
                "roofline_ms": roof_ms, "roofline_bound": "tensor" if flops / (tf * 1e12) > bytes_ / (hbm * 1e9) else "hbm",
                "roofline_frac": roof_ms / gemm_ms, "device_status": int(bufs.dev_status.item())})
    return res


def projection_only(log2_params, block, timer, reps):
    hbm, _, src = peaks()
    rows, cols = inputs.projection_sweep_shape(log2_params)
    wl = inputs.Workload(f"proj_2^{log2_params}_b{block}", 5, rows, cols, block, 500, 250, 0.02, m=0)
    ku = B.mwu_count_from_permille(wl.n_blocks, 500)
    kp = B.mwu_count_from_permille(wl.n_blocks, 250)
    desc = B.make_desc(rows, cols, block, ku, kp)
    W = inputs.normal_weights(rows, cols, 0.02, inputs.seed_for(5, 900 + log2_params)).cuda()
    bufs = B.ProjectionBuffers(desc, want_q=True)
    for _ in range(2):
        bufs.project(W)
    torch.cuda.synchronize()
    ms, best = timer.time(lambda: bufs.project(W), reps)
    return {"workload": wl.name, "rows": rows, "cols": cols, "block": block, "project_ms": ms,
            "project_best_ms": best, "projection_gbs_algorithmic": 8.0 * rows * cols / (ms * 1e-3) / 1e9,
            "projection_frac_of_hbm": 8.0 * rows * cols / (ms * 1e-3) / 1e9 / hbm, "peaks": src,
            "device_status": int(bufs.dev_status.item())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--set", default="main", choices=["main", "blocks", "projection", "all"])
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--only", default="", help="run just this workload of the main set")
    ap.add_argument("--m", type=int, default=0, help="override the activation rows of linear workloads")
    ap.add_argument("--fused", action="store_true", help="never use the decode-once workspace path")
    args = ap.parse_args()
    B.lib()
    timer = Timer()
    if args.set in ("main", "all"):
        for name in ([args.only] if args.only else ["c1_linear", "c2_conv3x3", "c3_conv1x1", "c4_ffn"]):
            print(json.dumps(run_workload(inputs.WORKLOADS[name], timer, args.reps, args.m or None, args.fused)),
                  flush=True)
    if args.set in ("blocks", "all"):
        for b in (2, 4, 8, 16):
            for pr in (0, 250, 500, 750, 900):
                print(json.dumps(run_workload(inputs.sweep_workload(b, pr), timer, args.reps, None, args.fused)),
                      flush=True)
    if args.set in ("projection", "all"):
        for lg in (20, 22, 24, 26, 28):
            for b in (4, 16):
                print(json.dumps(projection_only(lg, b, timer, args.reps)), flush=True)


if __name__ == "__main__":
    main()
