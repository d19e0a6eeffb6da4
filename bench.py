#!/usr/bin/env python
"""Benchmark of the hot path: mwu_project -> mwu_pack -> mwu_gemm (or mwu_conv_implicit).

One "step" is one pass of the whole path over one weight tensor and one activation batch.
The headline value is the effective throughput of the step: surviving-block FLOPs of the GEMM
(2 * M * block * (blocks - pruned blocks)) divided by the time of the whole step, so the
projection and packing time are charged to it.  Per-phase numbers, the roofline of the
dominant kernel, the dense bf16 library routine on the same shape and the CPU checker's speed are
reported alongside.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Workloads: c1_linear, c2_conv3x3 (through mwu_conv_implicit), c3_conv1x1, c4_ffn (default),
c5_sweep_b{2,4,8,16}_p{0,250,500,750,900}, and the projection-only size sweep proj_p{20..28}_b{2,4,8,16}
(2^p weights; metric GB/s).  --prune-group RxC switches a linear workload to grouped pruning
(whole R x C groups of weights are pruned, counts rounded down to whole groups).
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
L2_BYTES = 126 * 1024 * 1024
FLUSH_BYTES = 256 * 1024 * 1024


def recorded_traffic(workload: str):
    """DRAM bytes per call of the product kernels, from the ncu captures summarised in
    profiles/dram_traffic.txt; None when the table has no row for the workload or the sources of
    those kernels have changed since the capture (the row names them and carries their digest)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        cells = [c.strip() for c in ln.strip().strip("|").split("|")]
        if len(cells) != 5 or cells[0] != workload or not cells[2].isdigit():
            continue
        h = hashlib.sha256()
        try:
            for name in cells[4].split():
                h.update(name.encode())
                h.update(open(os.path.join(ROOT, "paper_2106_08301_b200", "csrc", name), "rb").read())
        except OSError:
            return None
        return int(cells[2]) if h.hexdigest()[:16] == cells[3] else None
    return None


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
    if name.startswith("proj_p"):
        lg, b = name[len("proj_p"):].split("_b")
        return inputs.projection_sweep_workload(int(lg), int(b))
    raise SystemExit(f"unknown workload {name}")


def counts_for(wl, count_fn, group=None):
    mb = wl.n_blocks
    ku, kp = count_fn(mb, wl.unified_permille), count_fn(mb, wl.pruned_permille)
    if group is not None:
        per = group[0] * group[1] // wl.block            # blocks per prune group: whole groups only
        kp = kp // per * per
    return ku, kp


def effective_flops(wl, m, k_prune):
    return 2.0 * m * wl.block * (wl.n_blocks - k_prune)


def gemm_rows(wl, m_override=0):
    if wl.conv is not None:
        n, c, h, w, kh, kw, stride, pad = wl.conv
        return n * ((h + 2 * pad - kh) // stride + 1) * ((w + 2 * pad - kw) // stride + 1)
    return m_override if m_override > 0 else wl.m


def algorithmic_bytes(wl, m, k_unify, k_prune):
    """What the method itself must move: projection reads W and writes Q (8 B / weight);
    GEMM reads X, writes Y (bf16) and reads the compact packed weights."""
    mb = wl.n_blocks
    n_u, n_d = k_unify - k_prune, mb - k_unify
    packed_bits = 2 * k_prune + n_u * (32 + wl.block + 2) + n_d * (16 * wl.block + 2)
    x_bytes = 2.0 * m * wl.cols
    if wl.conv is not None:
        n, c, h, w = wl.conv[:4]
        x_bytes = 2.0 * n * c * h * w                      # the input image, not its lowered matrix
    return {"projection": 8.0 * wl.rows * wl.cols,
            "gemm": x_bytes + 2.0 * m * wl.rows + packed_bits / 8.0}


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
            time.sleep(0.005)

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
def oracle_step(wl, w_rows: int, m_rows: int, group=None):
    """One pass of the path with the CPU checker on a bounded sample: the first w_rows rows of
    the weight (projection, storage form, decode) and the first m_rows activation rows (GEMM; for
    the convolution the first m_rows images)."""
    from oracle import mwu_oracle as O
    W = wl.weights()[:w_rows].numpy()
    mb = W.size // wl.block
    ku = O.count_from_permille(mb, wl.unified_permille)
    kp = O.count_from_permille(mb, wl.pruned_permille)
    if group is not None:
        per = group[0] * group[1] // wl.block
        kp = kp // per * per
    t0 = time.perf_counter()
    p = O.project(W, wl.block, ku, kp, prune_group=group)
    t1 = time.perf_counter()
    O.pack(p)
    t2 = time.perf_counter()
    What = O.decoded_weights(p)
    flops, checksum = 0.0, 0.0
    if wl.conv is not None:
        n, c, h, w, kh, kw, stride, pad = wl.conv
        x = wl.activations()[:m_rows].to(torch.float64).numpy()
        y = O.conv2d_direct(x, What, kh, kw, stride, pad)
        flops = 2.0 * y.shape[0] * y.shape[2] * y.shape[3] * wl.block * (mb - kp)
        checksum = float(np.abs(y).sum())
    elif wl.m > 0:
        X = wl.activations(m=m_rows).to(torch.float64).numpy()
        Y = O.gemm(X, What)
        flops = 2.0 * m_rows * wl.block * (mb - kp)
        checksum = float(np.abs(Y).sum())
    t3 = time.perf_counter()
    return {"seconds": t3 - t0, "project_s": t1 - t0, "pack_s": t2 - t1, "gemm_s": t3 - t2,
            "flops": flops, "params": W.size, "checksum": checksum}


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_sizes(wl, seconds: float, group=None):
    """Rows of W and of the activations for about `seconds` of checker work: a probe on 1/32 of
    the weight rows gives the rate (the work is linear in both counts)."""
    step_r = group[0] if group is not None else 1
    m_full = wl.conv[0] if wl.conv is not None else max(wl.m, 0)
    probe_r = max(step_r, min(wl.rows, max(8, wl.rows // 32) // step_r * step_r))
    probe_m = max(1, min(m_full, max(1, m_full // 32))) if m_full else 0
    t = oracle_step(wl, probe_r, probe_m, group)["seconds"]
    full_est = t * (wl.rows / probe_r) * ((m_full / probe_m) if probe_m else 1.0) ** 0.5
    if full_est <= seconds:
        return wl.rows, m_full
    # shrink both counts by the same factor f: the projection scales with f, the GEMM with f^2
    f = max(1.0 / 32, min(1.0, seconds / max(t * 32, 1e-9)))
    rows = max(probe_r, int(wl.rows * f) // step_r * step_r)
    return rows, (max(probe_m, int(m_full * f)) if m_full else 0)


def sample_text(wl, w_rows, m_rows, r=None):
    unit = "images" if wl.conv is not None else "activation rows"
    m_full = wl.conv[0] if wl.conv is not None else wl.m
    s = f"CPU checker as it stands: first {w_rows} of {wl.rows} weight rows (project, storage form, decode)"
    if m_full:
        s += f" and {m_rows} of {m_full} {unit} (fp64 GEMM / direct convolution) per step"
    if r is not None:
        s += f"; project {r['project_s']:.2f} s, pack {r['pack_s']:.2f} s, decode + product {r['gemm_s']:.2f} s"
    return s


def parse_group(text):
    if not text:
        return None
    r, c = text.lower().split("x")
    return int(r), int(c)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = get_workload(args.workload)
    group = parse_group(args.prune_group)
    steps, warm = max(1, args.steps), max(0, args.warmup)
    w_rows, m_rows = oracle_sample_sizes(wl, 120.0 / (steps + warm), group)
    for _ in range(warm):
        oracle_step(wl, w_rows, m_rows, group)
    t0 = time.perf_counter()
    flops, params = 0.0, 0.0
    for _ in range(steps):
        r = oracle_step(wl, w_rows, m_rows, group)
        flops += r["flops"]
        params += r["params"]
    dt = time.perf_counter() - t0
    proj_only = wl.m == 0 and wl.conv is None
    value = (8.0 * params / dt / 1e9) if proj_only else flops / dt / 1e12
    unit = "GB/s" if proj_only else UNIT
    line = {"impl": "reference", "metric": "mwu_projection_gbs" if proj_only else METRIC, "value": value,
            "unit": unit, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, None, None, gemm_rows(wl, args.m), group),
            "cpu_baseline": {"value": value, "unit": unit, "cores": cpu_threads(), "kind": "oracle",
                             "sample": sample_text(wl, w_rows, m_rows)},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def config_of(wl, ku, kp, m, group):
    cfg = {"workload": wl.name, "rows": wl.rows, "cols": wl.cols, "block": wl.block,
           "unified_permille": wl.unified_permille, "pruned_permille": wl.pruned_permille, "m": m}
    if group is not None:
        cfg["prune_group"] = f"{group[0]}x{group[1]}"
    return cfg


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
    group = parse_group(args.prune_group)
    is_conv = wl.conv is not None
    proj_only = wl.m == 0 and not is_conv
    m = gemm_rows(wl, args.m)
    ku, kp = counts_for(wl, B.mwu_count_from_permille, group)
    desc = B.make_desc(wl.rows, wl.cols, wl.block, ku, kp, prune_group=group)
    W_host = wl.weights().pin_memory()
    W = W_host.cuda()
    bufs = B.ProjectionBuffers(desc, want_q=True)
    stream = torch.cuda.current_stream()
    X_host = X = Y = Y_host = packed = workspace = None
    ws_bytes = 0
    if not proj_only:
        X_host = (wl.activations() if is_conv else wl.activations(m=m)).pin_memory()
        X = X_host.cuda()
        packed = torch.empty(B.mwu_packed_bytes(desc), dtype=torch.uint8, device="cuda")
        if is_conv:
            n, c, h, w, kh, kw, stride, pad = wl.conv
            oh, ow = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
            Y = torch.empty((n, wl.rows, oh, ow), dtype=torch.bfloat16, device="cuda")
            ws_bytes = 0 if args.fused else B.mwu_conv_workspace_bytes(desc, n, c, h, w, kh, kw, stride, pad)
        else:
            Y = torch.empty((m, wl.rows), dtype=torch.bfloat16, device="cuda")
            ws_bytes = 0 if args.fused else B.mwu_gemm_workspace_bytes(desc, m)
        Y_host = torch.empty(Y.shape, dtype=torch.bfloat16).pin_memory()
        workspace = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None

    def product(Xd, Yd, st):
        if is_conv:
            n, c, h, w, kh, kw, stride, pad = wl.conv
            B.mwu_conv_implicit_ws(desc, packed, Xd, n, c, h, w, kh, kw, stride, pad, Yd, 0, workspace,
                                   bufs.dev_status, stream=st)
        else:
            B.mwu_gemm_ws(desc, packed, Xd, m, wl.cols, Yd, wl.rows, 0, workspace, bufs.dev_status, stream=st)

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
        if not proj_only:
            bufs.pack(Wd, packed=packed, stream=st)
        if events is not None:
            events[2].record(st)
        if not proj_only:
            product(Xd, Yd, st)
        if events is not None:
            events[3].record(st)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # the step's inputs and outputs against L2: larger ones evict themselves, smaller ones get a
    # 256 MB write between the timed steps
    touched = W.numel() * 8 + (0 if proj_only else X.numel() * 2 + Y.numel() * 2)
    flush = touched <= 2 * L2_BYTES
    flush_buf = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda") if flush else None

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    if int(bufs.dev_status.item()) != 0:
        raise SystemExit(f"device status {int(bufs.dev_status.item())} after warm-up")

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    launches0 = B.mwu_kernel_launches()
    barrier()
    sampler.start()
    t_begin.record(stream)
    for i in range(args.steps):
        if flush:
            flush_buf.fill_(i & 0xff)
        step(ev[i])
    t_end.record(stream)
    barrier()
    sampler.stop()
    launches = B.mwu_kernel_launches() - launches0
    if flush:
        # the flush writes sit between the steps: the step time is the sum of the per-step event pairs
        total_ms = sum(e[0].elapsed_time(e[3]) for e in ev)
    else:
        total_ms = t_begin.elapsed_time(t_end)
    total_ms = replicas.max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    proj_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    pack_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    gemm_ms = statistics.mean(e[2].elapsed_time(e[3]) for e in ev)
    status = int(bufs.dev_status.item())

    # End to end through the C ABI with host buffers: every step copies its W and X from pinned host
    # memory and its result back (Y; for a projection-only workload Q).  The copies run on their own
    # streams with two sets of device buffers, so step i's download and step i+1's upload overlap step
    # i's kernels (the link is full duplex); the kernels themselves stay in order on one stream and
    # share the projection / packed buffers.
    e2e_steps = max(2, min(args.steps, 30))
    Wb = [W, torch.empty_like(W)]
    Xb = [X, torch.empty_like(X)] if X is not None else [None, None]
    if proj_only:
        out_dev = [bufs.Q, bufs.Q]
        out_host = [torch.empty(bufs.Q.shape, dtype=torch.float32).pin_memory() for _ in range(2)]
    else:
        out_dev = [Y, torch.empty_like(Y)]
        out_host = [Y_host, torch.empty_like(Y_host).pin_memory()]
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
            if X is not None:
                Xb[b].copy_(X_host, non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        if i >= (1 if proj_only else 2):
            stream.wait_event(ev_out[b if not proj_only else 1 - b])   # the output buffer has been downloaded
        step(None, Wb[b], Xb[b], out_dev[b] if not proj_only else None, stream)
        ev_comp[b].record(stream)
        s_out.wait_event(ev_comp[b])
        with torch.cuda.stream(s_out):
            out_host[b].copy_(out_dev[b], non_blocking=True)
            ev_out[b].record(s_out)
    stream.wait_event(ev_out[0])
    stream.wait_event(ev_out[1])
    t1.record(stream)
    barrier()
    e2e_ms = replicas.max_over_ranks(t0.elapsed_time(t1) / e2e_steps, dist, "cuda")
    h2d = W.numel() * 4 + (X.numel() * 2 if X is not None else 0)
    d2h = out_dev[0].numel() * out_dev[0].element_size()
    del Wb, Xb

    abytes = algorithmic_bytes(wl, m, ku, kp)
    peaks = measured_peaks()
    if proj_only:
        units, scale, metric, unit = abytes["projection"], 1e9, "mwu_projection_gbs", "GB/s"
    else:
        units, scale, metric, unit = effective_flops(wl, m, kp), 1e12, METRIC, UNIT
    value = replicas.whole_job_rate(units, world, ms_per_step) / scale
    e2e_value = replicas.whole_job_rate(units, world, e2e_ms) / scale

    cfg = config_of(wl, ku, kp, m, group)
    cfg.update({"k_unify": ku, "k_prune": kp, "parallelism": "replicas only",
                "l2": ("a 256 MB write between the timed steps (step time = sum of per-step event pairs)"
                       if flush else "inputs and outputs larger than L2 (%.0f MB touched per step)" % (touched / 1e6))})
    if not proj_only:
        cfg["product_path"] = (("weights expanded once per call (workspace %.1f MB), then a two-operand tensor-core kernel"
                                % (ws_bytes / 1e6)) if ws_bytes else "decode fused into the tensor-core kernel")
    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64" if proj_only else "bf16", "data": "synthetic",
        "config": cfg, "gpu_launches": int(launches), "device_status": status,
    }
    if rank == 0:
        proj_gbs = abytes["projection"] / (proj_ms * 1e-3) / 1e9
        phases = {"project_ms": proj_ms, "pack_ms": pack_ms, "product_ms": gemm_ms,
                  "projection_gbs_algorithmic": proj_gbs}
        roof_proj = {"bound": "hbm", "achieved": proj_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": proj_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy)",
                     "algorithmic_bytes_per_launch": abytes["projection"], "traffic": None,
                     "what": "the whole mwu_project call against the 8 bytes per weight the method needs"}
        if proj_only:
            line["roofline"] = dict(roof_proj, kernel="mwu_project (all its kernels)")
        else:
            flops = effective_flops(wl, m, kp)
            dense_flops = 2.0 * m * wl.rows * wl.cols
            # the dense bf16 library routine on the same shape (decoded weights), same process
            Wq = bufs.Q.reshape(wl.rows, wl.cols).to(torch.bfloat16)
            if is_conv:
                n, c, h, w, kh, kw, stride, pad = wl.conv
                Wq4 = Wq.reshape(wl.rows, c, kh, kw)
                lib = lambda: torch.nn.functional.conv2d(X, Wq4, stride=stride, padding=pad)
            else:
                lib = lambda: torch.matmul(X, Wq.T)
            for _ in range(3):
                lib()
            lib_ms = []
            for i in range(10):
                if flush:
                    flush_buf.fill_(i)
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record()
                lib()
                c1.record()
                torch.cuda.synchronize()
                lib_ms.append(c0.elapsed_time(c1))
            lib_ms = statistics.median(lib_ms)
            t_flops = flops / (peaks["bf16_tflops"] * 1e12)
            t_bytes = abytes["gemm"] / (peaks["hbm_gbs"] * 1e9)
            bound = "tensor" if t_flops >= t_bytes else "hbm"
            eff = flops / (gemm_ms * 1e-3) / 1e12
            phases.update({
                "product_effective_tflops": eff,
                "product_executed_dense_tflops": dense_flops / (gemm_ms * 1e-3) / 1e12,
                "executed_over_effective": dense_flops / flops,
                "library_dense_bf16_ms": lib_ms,
                "library_dense_bf16_tflops": dense_flops / (lib_ms * 1e-3) / 1e12,
                "decode_round_trip_bytes": 2 * ws_bytes,
                "note": ("effective counts surviving-block FLOPs only; executed_dense counts what the tensor "
                         "cores run when nothing can be skipped.  Per-block pruning with an iid pattern leaves no "
                         "dead tile slice, so the effective fraction of the tensor peak is capped near "
                         "(1 - pruned fraction) x (dense rate / peak)"),
                "dense_execution_ceiling_frac": (flops / dense_flops) * min(
                    1.0, dense_flops / (lib_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]),
            })
            if bound == "tensor":
                roof = {"bound": "tensor", "achieved": eff, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                        "frac": eff / peaks["bf16_tflops"],
                        "peak_source": peaks["source"] + " (cuBLAS bf16, burst: the kernel is timed in a run of milliseconds at full clocks)",
                        "frac_of_sustained_peak": eff / peaks["bf16_tflops_sustained"],
                        "sustained_peak": peaks["bf16_tflops_sustained"],
                        "algorithmic_flops_per_launch": flops}
            else:
                gbs = abytes["gemm"] / (gemm_ms * 1e-3) / 1e9
                roof = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy)",
                        "algorithmic_bytes_per_launch": abytes["gemm"]}
            roof["kernel"] = ("mwu_conv_implicit" if is_conv else "mwu_gemm") + (
                " (decode kernel + two-operand tensor-core kernel, timed together)" if ws_bytes else " (fused kernel)")
            roof["roofline_ms"] = max(t_flops, t_bytes) * 1e3
            # DRAM bytes come from an ncu capture of this call, not from this run; null once the kernels changed
            roof["traffic"] = recorded_traffic(wl.name) if (ws_bytes and not args.m and not group) else None
            roof["traffic_source"] = ("ncu capture of this call (dram__bytes_read.sum + dram__bytes_write.sum), recorded "
                                      "with a digest of the kernels' sources; the digest still matches"
                                      if roof["traffic"] is not None else
                                      "none: no capture recorded for this workload and launch configuration, or the "
                                      "kernels changed since it was taken")
            roof["projection"] = roof_proj
            line["roofline"] = roof
            if not is_conv and W.numel() >= (1 << 22):
                # the fused ADMM step (projection + dual update + quadratic term) on the same weight with a
                # dual tensor, timed beside the path: 16 bytes per weight are what it has to move
                U_dual = torch.randn(W.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(21060830)) * 0.004
                U_next = torch.empty(W.numel(), dtype=torch.float32, device="cuda")
                resid = torch.zeros(1, dtype=torch.float64, device="cuda")
                for _ in range(3):
                    bufs.admm_step(W, U_dual, U_next, resid)
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a0.record()
                for _ in range(20):
                    bufs.admm_step(W, U_dual, U_next, resid)
                a1.record()
                torch.cuda.synchronize()
                admm_ms = a0.elapsed_time(a1) / 20
                del U_dual, U_next
                phases["admm_step_ms"] = admm_ms
                gbs = 16.0 * W.numel() / (admm_ms * 1e-3) / 1e9
                roof["admm_step"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                     "frac": gbs / peaks["hbm_gbs"],
                                     "what": "mwu_admm_step: W, U in; Q, U_next out (16 bytes per weight)"}
        line["phases"] = phases
        line["clocks"] = sampler.summary()
        line["e2e"] = {"value": e2e_value, "unit": unit, "ms_per_step": e2e_ms, "steps": e2e_steps,
                       "overlap": "uploads, kernels and downloads on three streams, two buffer sets",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        if world == 1:
            w_rows, m_rows = oracle_sample_sizes(wl, 20.0, group)
            r = oracle_step(wl, w_rows, m_rows, group)
            cpu_units = 8.0 * r["params"] if proj_only else r["flops"]
            line["cpu_baseline"] = {
                "value": cpu_units / r["seconds"] / scale, "unit": unit, "cores": cpu_threads(),
                "kind": "oracle", "seconds": r["seconds"], "sample": sample_text(wl, w_rows, m_rows, r)}
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
                    help="no workspace: the product kernel decodes the packed weights inside its main loop")
    ap.add_argument("--prune-group", default="", help="RxC: prune whole groups of R rows x C columns")
    ap.add_argument("--impl", default="mwu", choices=["mwu", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
