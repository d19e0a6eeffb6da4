#!/usr/bin/env python
"""Benchmark of the hot path: mwu_project -> mwu_pack -> mwu_gemm on one synthetic workload.

One "step" is one pass of the whole path over one weight tensor and one activation batch.
The headline value is the effective throughput of the step: surviving-block FLOPs of the GEMM
(2 * M * block * (blocks - pruned blocks)) divided by the time of the whole step, so the
projection and packing time are charged to it.  Per-phase numbers, the roofline of the
dominant kernel, a cuBLAS dense bf16 comparison and the CPU checker's speed are reported
alongside.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4_ffn] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2106_08301_b200 import inputs, replicas  # noqa: E402

METRIC = "mwu_hot_path_effective_tflops"
UNIT = "TFLOP/s"
# launches per step: sample, pass, list_select, list_finish, then the four multi-pass kernels that
# return at once unless the one-pass result was given up (stats, prune_select, collect, emit)
# | count, scan, fill | gemm
KERNELS_PER_STEP = 12
KERNELS_PER_STEP_WS = 13  # ... | decode, dense gemm (with a workspace and enough activation rows)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def get_workload(name: str) -> inputs.Workload:
    if name in inputs.WORKLOADS:
        return inputs.WORKLOADS[name]
    if name.startswith("c5_sweep_b"):
        b, p = name[len("c5_sweep_b"):].split("_p")
        return inputs.sweep_workload(int(b), int(p))
    raise SystemExit(f"unknown workload {name}")


def counts_for(wl, count_fn):
    mb = wl.n_blocks
    return count_fn(mb, wl.unified_permille), count_fn(mb, wl.pruned_permille)


def effective_flops(wl, m, k_prune):
    return 2.0 * m * wl.block * (wl.n_blocks - k_prune)


def algorithmic_bytes(wl, m, k_unify, k_prune):
    """What the method itself must move: projection reads W and writes Q (8 B / weight);
    GEMM reads X, writes Y (bf16) and reads the compact packed weights."""
    mb = wl.n_blocks
    n_u, n_d = k_unify - k_prune, mb - k_unify
    packed_bits = 2 * k_prune + n_u * (32 + wl.block + 2) + n_d * (16 * wl.block + 2)
    return {"projection": 8.0 * wl.rows * wl.cols,
            "gemm": 2.0 * m * wl.cols + 2.0 * m * wl.rows + packed_bits / 8.0}


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _poll(self):
        while not self._stop.is_set():
            self.sample_once()
            time.sleep(0.01)

    def sample_once(self):
        if self.nv is None:
            return
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            r = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        self.sample_once()

    def summary(self):
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------------
# CPU checker timing (the reference arm and the cpu_baseline leg)
# ----------------------------------------------------------------------------------------------
def oracle_step(wl, W_rows: int, m_rows: int):
    """One pass of the path with the CPU checker on a bounded sample: the first W_rows rows of
    the weight (projection, packing, decode) and the first m_rows activation rows (GEMM)."""
    from oracle import mwu_oracle as O
    W = wl.weights()[:W_rows].numpy()
    X = wl.activations(m=m_rows).to(torch.float64).numpy()
    mb = W.size // wl.block
    ku = O.count_from_permille(mb, wl.unified_permille)
    kp = O.count_from_permille(mb, wl.pruned_permille)
    t0 = time.perf_counter()
    p = O.project(W, wl.block, ku, kp)
    t1 = time.perf_counter()
    O.pack(p, wl.block)
    t2 = time.perf_counter()
    Y = O.gemm(X, O.decoded_weights(p, wl.block))
    t3 = time.perf_counter()
    flops = 2.0 * m_rows * wl.block * (mb - kp)
    return {"seconds": t3 - t0, "project_s": t1 - t0, "pack_s": t2 - t1, "gemm_s": t3 - t2,
            "flops": flops, "params": W.size, "checksum": float(np.abs(Y).sum())}


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_sizes(wl):
    # about 10-30 s of CPU work on the default workload: all weight rows, up to 8192 activation rows
    return wl.rows, min(8192, max(1, wl.m))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = get_workload(args.workload)
    w_rows, m_rows = oracle_sample_sizes(wl)
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    for _ in range(warm):
        oracle_step(wl, w_rows, m_rows)
    t0 = time.perf_counter()
    flops = 0.0
    for _ in range(steps):
        r = oracle_step(wl, w_rows, m_rows)
        flops += r["flops"]
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = (f"CPU checker as it stands: first {w_rows} of {wl.rows} weight rows (project, pack, "
              f"decode) and {m_rows} of {wl.m} activation rows (fp64 GEMM) per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "rows": wl.rows, "cols": wl.cols, "block": wl.block,
                       "unified_permille": wl.unified_permille, "pruned_permille": wl.pruned_permille,
                       "m": wl.m},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------
def run_gpu(args):
    from paper_2106_08301_b200 import binding as B
    from paper_2106_08301_b200 import build as build_mod
    build_mod.build()
    B.lib()                                   # fail loudly if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod

    wl = get_workload(args.workload)
    if wl.conv is not None:
        raise SystemExit("bench.py times linear workloads; the convolution is timed by "
                         "paper_2106_08301_b200/sweep.py")
    m = args.m if args.m > 0 else wl.m
    ku, kp = counts_for(wl, B.mwu_count_from_permille)
    desc = B.make_desc(wl.rows, wl.cols, wl.block, ku, kp)
    W_host = wl.weights().pin_memory()
    X_host = wl.activations(m=m).pin_memory()
    W = W_host.cuda()
    X = X_host.cuda()
    bufs = B.ProjectionBuffers(desc, want_q=True)
    packed = torch.empty(B.mwu_packed_bytes(desc), dtype=torch.uint8, device="cuda")
    Y = torch.empty((m, wl.rows), dtype=torch.bfloat16, device="cuda")
    Y_host = torch.empty((m, wl.rows), dtype=torch.bfloat16).pin_memory()
    stream = torch.cuda.current_stream()
    ws_bytes = 0 if args.fused else B.mwu_gemm_workspace_bytes(desc, m)
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None

    def step(events=None, Wd=None, Xd=None, Yd=None, st=None):
        Wd = W if Wd is None else Wd
        Xd = X if Xd is None else Xd
        Yd = Y if Yd is None else Yd
        st = stream if st is None else st
        if events is not None:
            events[0].record(st)
        bufs.project(Wd, stream=st)
        if events is not None:
            events[1].record(st)
        bufs.pack(Wd, packed=packed, stream=st)
        if events is not None:
            events[2].record(st)
        B.mwu_gemm_ws(desc, packed, Xd, m, wl.cols, Yd, wl.rows, 0, workspace, bufs.dev_status, stream=st)
        if events is not None:
            events[3].record(st)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    if int(bufs.dev_status.item()) != 0:
        raise SystemExit(f"device status {int(bufs.dev_status.item())} after warm-up")

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t_begin.record(stream)
    for i in range(args.steps):
        step(ev[i])
    t_end.record(stream)
    barrier()
    sampler.stop()
    total_ms = replicas.max_over_ranks(t_begin.elapsed_time(t_end), dist, "cuda")
    ms_per_step = total_ms / args.steps
    proj_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    pack_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    gemm_ms = statistics.mean(e[2].elapsed_time(e[3]) for e in ev)
    status = int(bufs.dev_status.item())

    # End to end through the C ABI with host buffers: every step copies its W and X from pinned host
    # memory and its Y back.  The copies run on their own streams with two sets of device buffers,
    # so step i's download and step i+1's upload overlap step i's kernels (the link is full duplex);
    # the kernels themselves stay in order on one stream and share the projection / packed buffers.
    e2e_steps = max(2, min(args.steps, 30))
    Wb, Xb, Yb = [W, torch.empty_like(W)], [X, torch.empty_like(X)], [Y, torch.empty_like(Y)]
    Yh = [Y_host, torch.empty_like(Y_host).pin_memory()]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]       # upload of buffer set b done
    ev_comp = [torch.cuda.Event() for _ in range(2)]     # kernels on buffer set b done
    ev_out = [torch.cuda.Event() for _ in range(2)]      # download from buffer set b done
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    s_in.wait_event(t0)
    for i in range(e2e_steps):
        b = i % 2
        if i >= 2:
            s_in.wait_event(ev_comp[b])                  # the kernels of step i-2 have read W, X of this set
        with torch.cuda.stream(s_in):
            Wb[b].copy_(W_host, non_blocking=True)
            Xb[b].copy_(X_host, non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        if i >= 2:
            stream.wait_event(ev_out[b])                 # Y of this set has been downloaded
        step(None, Wb[b], Xb[b], Yb[b], stream)
        ev_comp[b].record(stream)
        s_out.wait_event(ev_comp[b])
        with torch.cuda.stream(s_out):
            Yh[b].copy_(Yb[b], non_blocking=True)
            ev_out[b].record(s_out)
    stream.wait_event(ev_out[0])
    stream.wait_event(ev_out[1])
    t1.record(stream)
    barrier()
    e2e_ms = replicas.max_over_ranks(t0.elapsed_time(t1) / e2e_steps, dist, "cuda")
    del Wb, Xb, Yb

    flops = effective_flops(wl, m, kp)
    dense_flops = 2.0 * m * wl.rows * wl.cols
    abytes = algorithmic_bytes(wl, m, ku, kp)
    peaks = measured_peaks()
    value = replicas.whole_job_rate(flops, world, ms_per_step) / 1e12
    e2e_value = replicas.whole_job_rate(flops, world, e2e_ms) / 1e12

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "rows": wl.rows, "cols": wl.cols, "block": wl.block,
                   "k_unify": ku, "k_prune": kp, "m": m, "parallelism": "replicas only",
                   "gemm_path": "decode once + two-operand GEMM (workspace %.0f MB)" % (ws_bytes / 1e6)
                   if ws_bytes else "decode fused into the GEMM",
                   "l2": "inputs larger than L2 (W %.0f MB, X %.0f MB, Y %.0f MB)" % (
                       W.numel() * 4 / 1e6, X.numel() * 2 / 1e6, Y.numel() * 2 / 1e6)},
        "gpu_launches": (KERNELS_PER_STEP_WS if ws_bytes else KERNELS_PER_STEP) * args.steps,
        "device_status": status,
    }
    if rank == 0:
        # cuBLAS dense bf16 on the same shape (decoded weights), same process
        Wd = bufs.Q.reshape(wl.rows, wl.cols).to(torch.bfloat16)
        for _ in range(3):
            torch.matmul(X, Wd.T)
        c0 = torch.cuda.Event(enable_timing=True)
        c1 = torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        c0.record()
        for _ in range(10):
            torch.matmul(X, Wd.T)
        c1.record()
        torch.cuda.synchronize()
        cublas_ms = c0.elapsed_time(c1) / 10
        # the fused ADMM step (projection + dual update + quadratic term) on the same weight with a
        # dual tensor, timed beside the path: 16 bytes per weight are what it has to move
        U_dual = torch.randn(W.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(21060830)) * 0.004
        U_next = torch.empty(W.numel(), dtype=torch.float32, device="cuda")
        resid = torch.zeros(1, dtype=torch.float64, device="cuda")
        for _ in range(3):
            bufs.admm_step(W, U_dual, U_next, resid)
        a0 = torch.cuda.Event(enable_timing=True)
        a1 = torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a0.record()
        for _ in range(20):
            bufs.admm_step(W, U_dual, U_next, resid)
        a1.record()
        torch.cuda.synchronize()
        admm_ms = a0.elapsed_time(a1) / 20
        del U_dual, U_next
        line["phases"] = {
            "project_ms": proj_ms, "pack_ms": pack_ms, "gemm_ms": gemm_ms,
            "projection_gbs_algorithmic": abytes["projection"] / (proj_ms * 1e-3) / 1e9,
            "gemm_effective_tflops": flops / (gemm_ms * 1e-3) / 1e12,
            "gemm_executed_dense_tflops": dense_flops / (gemm_ms * 1e-3) / 1e12,
            "admm_step_ms": admm_ms,
            "admm_step_gbs_algorithmic": 16.0 * W.numel() / (admm_ms * 1e-3) / 1e9,
            "cublas_dense_bf16_ms": cublas_ms,
            "cublas_dense_bf16_tflops": dense_flops / (cublas_ms * 1e-3) / 1e12,
        }
        peak_tf = peaks["bf16_tflops_sustained"]
        ach = flops / (gemm_ms * 1e-3) / 1e12
        line["roofline"] = {
            "kernel": "mwu_decode_kernel + mwu_dense_pair_kernel" if ws_bytes else "mwu_gemm_pair_kernel",
            "bound": "tensor", "achieved": ach, "peak": peak_tf,
            "unit": "TFLOP/s", "frac": ach / peak_tf,
            "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
            "algorithmic_flops_per_launch": flops,
            # dram__bytes_read.sum + dram__bytes_write.sum of one launch of the two-operand GEMM kernel
            # (610.1 MB + 250.0 MB, ncu capture of this workload; see profiles/step_kernels_c4_ffn.md);
            # not taken for other workloads or for the fused path
            "traffic": 860.1e6 if (ws_bytes and wl.name == "c4_ffn" and m == wl.m) else None,
            # the whole mwu_project call (eight launches) against the 8 bytes per weight the method needs
            "projection": {"bound": "hbm", "achieved": abytes["projection"] / (proj_ms * 1e-3) / 1e9,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": abytes["projection"] / (proj_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            # mwu_admm_step: W, U in; Q, U_next out
            "admm_step": {"bound": "hbm", "achieved": 16.0 * W.numel() / (admm_ms * 1e-3) / 1e9,
                          "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": 16.0 * W.numel() / (admm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        }
        line["clocks"] = sampler.summary()
        line["e2e"] = {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
                       "overlap": "uploads, kernels and downloads on three streams, two buffer sets",
                       "h2d_bytes_per_step": W.numel() * 4 + X.numel() * 2,
                       "d2h_bytes_per_step": Y.numel() * 2}
        if world == 1:
            w_rows, m_rows = oracle_sample_sizes(wl)
            r = oracle_step(wl, w_rows, m_rows)
            line["cpu_baseline"] = {
                "value": r["flops"] / r["seconds"] / 1e12, "unit": UNIT, "cores": cpu_threads(),
                "kind": "oracle", "seconds": r["seconds"],
                "sample": (f"first {w_rows} of {wl.rows} weight rows (project {r['project_s']:.2f} s, "
                           f"pack {r['pack_s']:.2f} s) and {m_rows} of {m} activation rows "
                           f"(decode + fp64 GEMM {r['gemm_s']:.2f} s)")}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c4_ffn")
    ap.add_argument("--m", type=int, default=0, help="override the number of activation rows")
    ap.add_argument("--fused", action="store_true",
                    help="no workspace: the GEMM decodes the packed weights inside its main loop")
    ap.add_argument("--impl", default="mwu", choices=["mwu", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
