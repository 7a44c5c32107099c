#!/usr/bin/env python
"""Benchmark of the Attention Pruning path on B200.

One step = one pass of the whole path over one batch of synthetic input, all
through the C ABI: ap_accumulate_attention (one calibration batch) ->
ap_build_mask (mask + tile list) -> ap_sparse_attention_fwd under that mask ->
the library's dense path at the same shape (ap_dense_tiles + the same forward
kernel).  Prints ONE JSON line (rank 0).

  metric / value   effective TFLOP/s of the sparse forward, 4*d*nnz FLOPs per
                   (b, h), over the forward's device time inside the steps
  ms_per_step      the whole step (all four stages)
  e2e              the same metric through ap_sparse_attention_fwd_host: pinned
                   host Q, K, V in, O back, copies inside the timed region
  roofline         the forward kernel: executed tile FLOPs / time vs the
                   measured bf16 peak; `by_stage` gives the other stages
  cpu_baseline     the oracle (plain fp64 C) timed on a bounded sample

The path does not shard (single-GPU method): --gpus N runs N independent
replicas, one per GPU, and adds their throughput ("replicas only").

--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2012_02030_b200 import inputs, metrics, replicas  # noqa: E402

METRIC = "sparse-attention fwd effective TFLOP/s (4*d*nnz)"
UNIT = "TFLOP/s"

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each stage's kernels, from ncu
# captures of a REDUCED case of the same workload (fewer batch elements, so that the capture is small),
# scaled to the full launch by the units it processes; `source` says which capture and how it was scaled.
# A stage without a capture reports null.
NCU_TRAFFIC = {
    "long": {
        "sparse_fwd": {"bytes": 4 * 70.5e6,
                       "source": "ncu on the B=1 case (68.0 MB read + 2.5 MB written per launch), times 4 batch elements; "
                                 "O is still in L2 when the kernel ends"},
        "accumulate": {"bytes": 2.27e9,
                       "source": "ncu on the B=1 case (1.72 GB read + 0.50 GB written per launch: the accumulator, the bias "
                                 "and their traffic have no batch dimension) plus Q and K of three more samples"},
        "build_mask": {"bytes": 1.04e9,
                       "source": "ncu on the B=1 case (the accumulator and the mask have no batch dimension): the "
                                 "classifying pass 541 MB read + 304 MB written, the passes over the collected entries "
                                 "3 x 35 MB read, the patch pass 58 MB read + 13 MB written, the pivots' sample 17 MB read"},
    },
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p["bf16_tflops_sustained"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU while the timed steps run.

    Read-only NVML queries from a background thread every few milliseconds (the timed region of
    the default run lasts tens of milliseconds, too short for `nvidia-smi -lms`); falls back to
    an `nvidia-smi` child process where NVML cannot be loaded.  The device index is resolved
    through CUDA_VISIBLE_DEVICES when that holds plain indices.
    """

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_s: float = 0.001):
        import threading

        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x.strip() for x in vis.split(",") if x.strip()]
        if ids and all(x.isdigit() for x in ids) and gpu_index < len(ids):
            gpu_index = int(ids[gpu_index])
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self.proc = self.thread = None
        self._stop = threading.Event()
        try:
            import pynvml

            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            bits = {"hw_slowdown": pynvml.nvmlClocksEventReasonHwSlowdown,
                    "hw_thermal_slowdown": pynvml.nvmlClocksEventReasonHwThermalSlowdown,
                    "sw_thermal_slowdown": pynvml.nvmlClocksEventReasonSwThermalSlowdown,
                    "sw_power_cap": pynvml.nvmlClocksEventReasonSwPowerCap}

            def loop():
                while not self._stop.is_set():
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        r = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                        for name, bit in bits.items():
                            if r & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    time.sleep(period_s)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
        except Exception:
            try:
                self.proc = subprocess.Popen(
                    ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                     "--format=csv,noheader,nounits", "-lms", "20"],
                    stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            except OSError:
                self.proc = None

    def stop(self):
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
                    "samples": len(self.sm), "reasons": sorted(self.reasons), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["clock sampling unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi"}


# --------------------------------------------------------------------------- CPU oracle legs


def oracle_sample_step(w, units, calib_seqs=1, batch=1):
    """One pass of the path on the CPU oracle for a bounded sample: `units` heads, `calib_seqs`
    calibration sequences, the forward on `batch` batch elements.  Returns per-stage seconds and
    the FLOPs (4*d*nnz per batch element) of the forward."""
    from oracle import ap_oracle as orc

    heads = list(range(units))
    q, k = inputs.calib_qk(w, 0)
    bias = inputs.calib_bias(w)[heads].numpy()
    qs, ks = inputs.widen(q[:calib_seqs, heads]), inputs.widen(k[:calib_seqs, heads])
    acc64 = np.zeros((units, w.Lq, w.Lk))
    t0 = time.perf_counter()
    orc.accumulate(acc64, qs, ks, bias, causal=w.causal)
    t1 = time.perf_counter()
    mask, nnz = orc.build_mask(acc64.astype(np.float32), w.keep_frac, w.causal, w.keep_diag)
    t2 = time.perf_counter()
    eq, ek, ev = inputs.eval_qkv(w)
    eq, ek, ev = (inputs.widen(t[:batch, heads]) for t in (eq, ek, ev))
    t3 = time.perf_counter()
    orc.attention_fwd(eq, ek, ev, mask)
    t4 = time.perf_counter()
    flops = 4.0 * w.d * float(nnz.sum()) * batch
    return dict(acc_s=t1 - t0, mask_s=t2 - t1, fwd_s=t4 - t3, flops=flops, cores=min(orc.num_threads(), units))


def run_reference(args, w):
    """The oracle as it stands, on the host cores, on a bounded sample per step."""
    if replicas.rank_info().rank != 0:  # rank 0 alone runs the CPU arm
        return
    units = min(w.H, 8)
    for _ in range(args.warmup):
        oracle_sample_step(w, units)
    fwd_s, step_s, flops, cores = 0.0, 0.0, 0.0, 1
    for _ in range(args.steps):
        r = oracle_sample_step(w, units)
        fwd_s += r["fwd_s"]
        step_s += r["acc_s"] + r["mask_s"] + r["fwd_s"]
        flops += r["flops"]
        cores = r["cores"]
    value = flops / fwd_s / 1e12
    sample = "heads 0..%d of batch element 0 (%d of %d (b,h) units); one calibration sequence" % (
        units - 1, units, w.B * w.H)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * step_s / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w):
    return {"workload": w.name, "B": w.B, "H": w.H, "Lq": w.Lq, "Lk": w.Lk, "d": w.d, "causal": w.causal,
            "keep_frac": w.keep_frac, "keep_diag": w.keep_diag, "calib_batches": w.calib_batches,
            "replicas": "one per GPU, no exchange"}


# ------------------------------------------------------------------------------- GPU arm


def _stats(ms):
    ms = [float(x) for x in ms]
    return {"mean": float(np.mean(ms)), "median": float(np.median(ms)), "best": float(np.min(ms))}


def _time_back_to_back(fn, n):
    """n launches of fn(i) back to back between one pair of events: ms per launch."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def workloads_section(ap, dev, peaks, with_cpu):
    """Short runs of the small workloads: forward under the calibrated mask and under the dense list.
    Their tensors fit in L2, so the figure for the HBM roofline rotates over enough copies of the
    tensors to exceed L2 twice over (every launch finds its inputs in DRAM); the L2-warm figure (one
    set of tensors reused) is given beside it.  With with_cpu, the oracle's forward on a bounded
    sample is timed on one thread and on all threads."""
    out = {}
    for name in ("tiny", "bert", "lm", "s2s_self", "s2s_cross"):
        w = inputs.WORKLOADS[name]
        elem = 4 if w.dtype == "f32" else 2
        bias = inputs.calib_bias(w).to(dev)
        acc = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.float32, device=dev)
        for t in range(w.calib_batches):
            cq, ck = inputs.calib_qk(w, t)
            ap.ap_accumulate_attention(acc, cq.to(dev), ck.to(dev), bias, causal=w.causal)
        tiles = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
        dense = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
        nnz = torch.zeros((w.H,), dtype=torch.int64, device=dev)
        mask = torch.empty((w.H, w.Lq, w.Lk), dtype=torch.uint8, device=dev)
        ap.ap_build_mask(acc, w.keep_frac, w.causal, w.keep_diag, mask, tiles, nnz)
        ap.ap_dense_tiles(dense, causal=w.causal)
        q, k, v = (t.to(dev) for t in inputs.eval_qkv(w))
        set_bytes = 4 * q.numel() * elem
        n_sets = max(2, int(np.ceil(2.5 * 126e6 / set_bytes)))
        sets = [(q, k, v, torch.empty_like(q))] + [(q.clone(), k.clone(), v.clone(), torch.empty_like(q))
                                                   for _ in range(n_sets - 1)]
        n = max(20, 2 * n_sets)
        res = {}
        for label, tl in (("sparse", tiles), ("dense", dense)):
            for i in range(n_sets):   # warm-up: every set once
                ap.ap_sparse_attention_fwd(*sets[i][:3], tl, sets[i][3])
            cold = _time_back_to_back(lambda i: ap.ap_sparse_attention_fwd(*sets[i % n_sets][:3], tl, sets[i % n_sets][3]), n)
            warm = _time_back_to_back(lambda i: ap.ap_sparse_attention_fwd(*sets[0][:3], tl, sets[0][3]), n)
            res[label] = (cold, warm)
        if ap.ap_device_status() != ap.AP_OK:
            raise RuntimeError("device status not OK in the workloads section (%s)" % name)
        nnz_total = int(nnz.sum().item())
        comp = metrics.compulsory_bytes(w.B, w.H, w.Lq, w.Lk, w.d, elem)
        entry = {
            "shape": {"B": w.B, "H": w.H, "Lq": w.Lq, "Lk": w.Lk, "d": w.d, "dtype": w.dtype, "keep_frac": w.keep_frac,
                      "calib_batches": w.calib_batches},
            "sparse_fwd_ms": res["sparse"][0], "dense_fwd_ms": res["dense"][0],
            "sparse_fwd_ms_l2_warm": res["sparse"][1], "dense_fwd_ms_l2_warm": res["dense"][1],
            "speedup_vs_dense_path": res["dense"][0] / res["sparse"][0],
            "effective_tflops": metrics.effective_flops(nnz_total, w.B, w.d) / (res["sparse"][0] * 1e-3) / 1e12,
            "tokens_per_s": w.B * w.Lq / (res["sparse"][0] * 1e-3),
            "frac_of_hbm_on_compulsory_bytes": comp / (res["sparse"][0] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "tiles_kept": tiles.n_tiles(), "tiles_domain": dense.n_tiles(), "rounds": int(tiles.round_ptr[-1].item()),
            "buffer_sets": n_sets, "launches_timed": n,
        }
        if with_cpu:
            from oracle import ap_oracle as orc

            units, seqs = min(w.H, 4), min(w.B, 2)
            eq, ek, ev = (inputs.widen(t[:seqs, :units]) for t in inputs.eval_qkv(w))
            m_host = mask[:units].cpu().numpy()
            fl = 4.0 * w.d * float(m_host.sum()) * seqs
            all_threads = orc.num_threads()
            cpu = {}
            for label, nt in (("threads_1", 1), ("threads_all", all_threads)):
                orc.set_num_threads(nt)
                t0 = time.perf_counter()
                orc.attention_fwd(eq, ek, ev, m_host)
                cpu[label] = {"tflops": fl / (time.perf_counter() - t0) / 1e12, "threads": min(nt, units * seqs)}
            orc.set_num_threads(all_threads)
            cpu["sample"] = "oracle forward of heads 0..%d of batch elements 0..%d" % (units - 1, seqs - 1)
            entry["cpu_oracle"] = cpu
        out[name] = entry
        del sets, acc, mask, bias
    return out


def density_section(ap, w, acc, q, k, v, out, ws, dense_ms, dense_tiles, peaks, dev):
    """The forward on the bench's own shape and accumulator at several kept fractions: time, what the
    schedule holds, speedup over the dense list, fractions of the burst bf16 peak."""
    rows = []
    tiles = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    paired = ap.Tiles(w.H, w.Lq, w.Lk, device=dev, paired=True)  # units of work balanced by the list's builder
    nnz = torch.zeros((w.H,), dtype=torch.int64, device=dev)
    for keep in (0.10, 0.05, 0.02):
        ap.ap_build_mask(acc, keep, w.causal, w.keep_diag, None, paired, nnz, ws)
        for _ in range(3):
            ap.ap_sparse_attention_fwd(q, k, v, paired, out)
        ms_paired = _time_back_to_back(lambda i: ap.ap_sparse_attention_fwd(q, k, v, paired, out), 10)
        ap.ap_build_mask(acc, keep, w.causal, w.keep_diag, None, tiles, nnz, ws)
        for _ in range(3):
            ap.ap_sparse_attention_fwd(q, k, v, tiles, out)
        ms = _time_back_to_back(lambda i: ap.ap_sparse_attention_fwd(q, k, v, tiles, out), 10)
        n_rounds = int(tiles.round_ptr[-1].item())
        slots = int((tiles.round_info[:n_rounds] & 15).sum().item())
        n_tiles = tiles.n_tiles()
        kept = int(nnz.sum().item())
        rows.append({
            "keep_frac": keep, "kept_entries_per_head": kept // w.H, "fwd_ms": ms,
            "fwd_ms_with_balanced_units": ms_paired, "tiles": n_tiles, "rounds": n_rounds,
            "slots": slots, "speedup_vs_dense_path": dense_ms / ms,
            "effective_tflops": metrics.effective_flops(kept, w.B, w.d) / (ms * 1e-3) / 1e12,
            "frac_of_bf16_burst_on_kept_tile_flops": metrics.tile_flops(n_tiles, w.B, w.d) / (ms * 1e-3) / 1e12 / peaks["bf16"],
            "frac_of_bf16_burst_on_executed_flops": metrics.slot_flops(slots, w.B, w.d) / (ms * 1e-3) / 1e12 / peaks["bf16"],
        })
    if ap.ap_device_status() != ap.AP_OK:
        raise RuntimeError("device status not OK in the density section")
    return {"shape": w.name, "dense_path_ms": dense_ms, "dense_tiles": dense_tiles,
            "timing": "10 launches back to back after 3 warm-up launches; the tensors exceed L2", "rows": rows}

def gathered_section(ap, w, acc, q, k, v, out, ws, dev):
    """The tile list's second schedule (rounds of individually gathered key columns) against the rounds, on the
    bench's shape: under the method's own masks (where the builders' rule decides per list row) and under
    column-structured synthetic masks (single key columns shared by the rows of a query tile)."""
    rows = []
    tiles = ap.Tiles(w.H, w.Lq, w.Lk, device=dev, gathered=True)
    nnz = torch.zeros((w.H,), dtype=torch.int64, device=dev)

    def measure(label, build):
        row = {"mask": label}
        for mode, key in ((1, "rounds"), (0, "gathered_where_the_rule_allows"), (2, "gathered_everywhere")):
            ap.ap_debug_schedule(mode)
            try:
                build()
                for _ in range(3):
                    ap.ap_sparse_attention_fwd(q, k, v, tiles, out)
                row[key + "_ms"] = _time_back_to_back(lambda i: ap.ap_sparse_attention_fwd(q, k, v, tiles, out), 10)
            finally:
                ap.ap_debug_schedule(0)
            rp, gp = tiles.round_ptr.diff(), tiles.ground_ptr.diff()
            if mode == 1:
                row["rounds"] = int(rp.sum().item())
            else:
                row[key + "_rounds_followed"] = int(torch.where(gp > 0, gp, rp).sum().item())
                row[key + "_list_rows"] = int((gp > 0).sum().item())
        rows.append(row)

    for keep in (0.10, 0.05):
        measure("method's mask, keep %g" % keep,
                lambda: ap.ap_build_mask(acc, keep, w.causal, w.keep_diag, None, tiles, nnz, ws))
    gen = torch.Generator(device=dev).manual_seed(11)
    i = torch.arange(w.Lq, device=dev)[:, None]
    inside = (torch.arange(w.Lk, device=dev)[None, :] <= i + (w.Lk - w.Lq)) if w.causal else None
    for frac in (0.05, 0.3):
        sel = torch.rand((w.H, -(-w.Lq // 128), w.Lk), device=dev, generator=gen) < frac
        mask = sel.repeat_interleave(128, dim=1)[:, :w.Lq]
        if inside is not None:
            mask = mask & inside[None]
        mask = mask.to(torch.uint8)
        del sel
        measure("single columns per query tile, %g of the keys" % frac, lambda: ap.ap_mask_to_tiles(mask, tiles))
        del mask
    if ap.ap_device_status() != ap.AP_OK:
        raise RuntimeError("device status not OK in the gathered section")
    return {"shape": w.name, "list_rows": w.H * (-(-w.Lq // 128)),
            "timing": "10 launches back to back after 3 warm-up launches; the tensors exceed L2", "rows": rows}


def run_gpu(args, w):
    from paper_2012_02030_b200 import binding as ap

    info = replicas.rank_info()
    rank, local_rank, world = info.rank, info.local_rank, info.world
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init(info, "nccl", dev)
    peaks = load_peaks()
    elem = 4 if w.dtype == "f32" else 2

    # ---- resident inputs (host-generated, seeded) --------------------------------------
    bias = inputs.calib_bias(w).to(dev)
    # Calibration batches the steps add, one per step: distinct from the calibration set proper and
    # from one another (a few batches repeated over and over would come to dominate the running
    # sum and with it the mask the forward is timed on); they stay resident and are reused in turn
    # only when there are more steps than batches.
    n_rot = max(1, min(16, args.warmup + args.steps))
    calib = [tuple(t.to(dev) for t in inputs.calib_qk(w, w.calib_batches + r)) for r in range(n_rot)]
    q, k, v = (t.to(dev) for t in inputs.eval_qkv(w))
    out = torch.empty_like(q)
    out_dense = torch.empty_like(q)
    acc = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.float32, device=dev)
    mask = torch.empty((w.H, w.Lq, w.Lk), dtype=torch.uint8, device=dev)
    nnz = torch.zeros((w.H,), dtype=torch.int64, device=dev)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    dense = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    ws = torch.empty(ap.ap_build_mask_workspace_bytes(w.H, w.Lq, w.Lk), dtype=torch.uint8, device=dev)
    # small shapes: an L2 flush between steps; large ones exceed L2 by themselves
    resident = acc.numel() * 4 + bias.numel() * 4 + 4 * q.numel() * elem
    flush = None if resident > 400e6 else torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    # the calibration set proper (untimed): the mask the steps work with is the real one
    for t in range(args.calib_batches if args.calib_batches > 0 else w.calib_batches):
        cq, ck = inputs.calib_qk(w, t)
        ap.ap_accumulate_attention(acc, cq.to(dev), ck.to(dev), bias, causal=w.causal)
    torch.cuda.synchronize()

    t_log = torch.zeros((max(args.steps, 1),), dtype=torch.int32, device=dev)
    stages = ("accumulate", "build_mask", "sparse_fwd", "dense_tiles", "dense_fwd")

    def step(i, ev=None):
        cq, ck = calib[i % n_rot]
        if flush is not None:
            flush.zero_()
        if ev:
            ev[0].record()
        ap.ap_accumulate_attention(acc, cq, ck, bias, causal=w.causal)
        if ev:
            ev[1].record()
        ap.ap_build_mask(acc, w.keep_frac, w.causal, w.keep_diag, mask, tiles, nnz, ws)
        if ev:
            ev[2].record()
        ap.ap_sparse_attention_fwd(q, k, v, tiles, out)
        if ev:
            ev[3].record()
        ap.ap_dense_tiles(dense, causal=w.causal)
        if ev:
            ev[4].record()
        ap.ap_sparse_attention_fwd(q, k, v, dense, out_dense)
        if ev:
            ev[5].record()
            t_log[i].copy_(tiles.row_ptr[-1])

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if ap.ap_device_status() != ap.AP_OK:
        raise RuntimeError("device status not OK after warm-up")

    def barrier():
        replicas.barrier(info, dev)

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    launches0 = ap.ap_launch_count()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    barrier()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(args.steps):
        step(i, events[i])
    end.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    launches = ap.ap_launch_count() - launches0
    status = ap.ap_device_status()
    if status != ap.AP_OK:
        raise RuntimeError("device status %d after the timed steps" % status)
    total_ms = start.elapsed_time(end)
    stage_all = {s: _stats([events[i][j].elapsed_time(events[i][j + 1]) for i in range(args.steps)])
                 for j, s in enumerate(stages)}
    stage_ms = {s: stage_all[s]["mean"] for s in stages}
    total_ms, fwd_ms_max = replicas.max_over_ranks(info, [total_ms, stage_ms["sparse_fwd"]], dev)

    # ---- counts -----------------------------------------------------------------------------
    nnz_total = int(nnz.sum().item())
    k_expected = metrics.keep_count(w.n_valid, w.n_forced, w.keep_frac)
    assert nnz_total == k_expected * w.H, (nnz_total, k_expected)
    T_sparse = float(t_log[: args.steps].float().mean().item())
    T_dense = dense.n_tiles()
    # what the forward kernel executes: rounds of slots (non-empty groups of 16 key columns)
    n_rounds = int(tiles.round_ptr[-1].item())
    n_slots = int((tiles.round_info[:n_rounds] & 15).sum().item())
    eff_flops = metrics.effective_flops(nnz_total, w.B, w.d)
    value = replicas.job_throughput(info, eff_flops, fwd_ms_max * 1e-3) / 1e12

    # ---- end to end through host buffers ---------------------------------------------------------
    hq, hk, hv = (t.pin_memory() for t in inputs.eval_qkv(w))
    ho = torch.empty_like(hq).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        ap.ap_sparse_attention_fwd_host(hq, hk, hv, tiles, ho, q, k, v, out)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        ap.ap_sparse_attention_fwd_host(hq, hk, hv, tiles, ho, q, k, v, out)
        torch.cuda.current_stream().synchronize()  # the caller reads O on the host every step
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    (e2e_ms,) = replicas.max_over_ranks(info, [e2e_ms], dev)
    h2d = 3 * 0 + (hq.numel() + hk.numel() + hv.numel()) * elem
    d2h = ho.numel() * elem

    # ---- Eq. 2 with one threshold for the layer (outside the step: the workloads prescribe per head) ----
    tiles_layer = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    nnz_layer = torch.zeros((w.H,), dtype=torch.int64, device=dev)
    layer_ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    layer_ms = [0.0, 0.0]
    n_layer = 5
    for it in range(2 + n_layer):
        layer_ev[0].record()
        ap.ap_build_mask_layer(acc, w.keep_frac, w.causal, w.keep_diag, mask, tiles_layer, nnz_layer, ws)
        layer_ev[1].record()
        ap.ap_sparse_attention_fwd(q, k, v, tiles_layer, out)
        layer_ev[2].record()
        torch.cuda.synchronize()
        if it >= 2:
            layer_ms[0] += layer_ev[0].elapsed_time(layer_ev[1]) / n_layer
            layer_ms[1] += layer_ev[1].elapsed_time(layer_ev[2]) / n_layer
    if ap.ap_device_status() != ap.AP_OK:
        raise RuntimeError("device status not OK after the layer-threshold runs")
    k_layer = metrics.keep_count(w.n_valid * w.H, w.n_forced * w.H, w.keep_frac)
    assert int(nnz_layer.sum().item()) == k_layer
    layer = {"build_mask_layer_ms": layer_ms[0], "sparse_fwd_ms": layer_ms[1], "tiles_kept": tiles_layer.n_tiles(),
             "nnz_per_head_min": int(nnz_layer.min().item()), "nnz_per_head_max": int(nnz_layer.max().item()),
             "effective_tflops": metrics.effective_flops(k_layer, w.B, w.d) / (layer_ms[1] * 1e-3) / 1e12,
             "note": "one threshold over all heads of the layer; %d runs after 2 warm-up runs, outside the step"
                     % n_layer}

    # ---- derivative of the masked attention under the step's mask (outside the step) ----
    backward = None
    if w.dtype != "f32":
        gen = torch.Generator(device="cpu")
        gen.manual_seed(w.seed0 + 77)
        d_out = torch.randn(q.shape, generator=gen).to(q.dtype).to(dev)
        ap.ap_sparse_attention_fwd(q, k, v, tiles, out)
        grads = ap.ap_sparse_attention_bwd(q, k, v, out, d_out, tiles)
        bws = torch.empty(ap.ap_sparse_attention_bwd_workspace_bytes(w.B, w.H, w.Lq, w.Lk), dtype=torch.uint8, device=dev)
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_bwd = 5
        torch.cuda.synchronize()
        b0.record()
        for _ in range(n_bwd):
            ap.ap_sparse_attention_bwd(q, k, v, out, d_out, tiles, *grads, workspace=bws)
        b1.record()
        torch.cuda.synchronize()
        if ap.ap_device_status() != ap.AP_OK:
            raise RuntimeError("device status not OK after the backward runs")
        bwd_ms = b0.elapsed_time(b1) / n_bwd
        # executed (upper bound): the rows kernel works on rounds, four products per slot (S twice, dP, dQ:
        # 128 rows x 16 columns x d each); the columns kernel on stored tiles, four 128 x 128 x d products
        # per tile (S, dP over the span of non-empty groups at most, dV, dK in full);
        # effective: 10*d per kept entry (2.5 x the forward's 4*d)
        n_rounds_b = int(tiles.round_ptr[-1].item())
        n_slots_b = int((tiles.round_info[:n_rounds_b] & 15).sum().item())
        bwd_fl = (4 * 2.0 * 128 * 16 * w.d * n_slots_b + 4 * 2.0 * 128 * 128 * w.d * tiles.n_tiles()) * w.B
        backward = {"ms": bwd_ms, "effective_tflops": 10.0 * w.d * float(nnz.sum().item()) * w.B / (bwd_ms * 1e-3) / 1e12,
                    "executed_tflops": bwd_fl / (bwd_ms * 1e-3) / 1e12,
                    "frac_of_bf16_burst": bwd_fl / (bwd_ms * 1e-3) / 1e12 / peaks["bf16"],
                    "frac_of_bf16_sustained": bwd_fl / (bwd_ms * 1e-3) / 1e12 / peaks["bf16_sustained"],
                    "note": "ap_sparse_attention_bwd (rows kernel on rounds + columns kernel on tiles), %d runs "
                            "outside the step" % n_bwd}

    # ---- the same two stages for a model normalised by 1.5-entmax (outside the step) ----
    entmax = None
    if w.dtype != "f32":
        acc_e = torch.zeros_like(acc)
        cq, ck = calib[0]
        n_ent = 3
        ent_ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ent_ms = [0.0, 0.0]
        for it in range(2 + n_ent):
            ent_ev[0].record()
            ap.ap_accumulate_attention_entmax15(acc_e, cq, ck, bias, causal=w.causal)
            ent_ev[1].record()
            ap.ap_sparse_attention_entmax15_fwd(q, k, v, tiles, out)
            ent_ev[2].record()
            torch.cuda.synchronize()
            if it >= 2:
                ent_ms[0] += ent_ev[0].elapsed_time(ent_ev[1]) / n_ent
                ent_ms[1] += ent_ev[1].elapsed_time(ent_ev[2]) / n_ent
        if ap.ap_device_status() != ap.AP_OK:
            raise RuntimeError("device status not OK after the entmax runs")
        support = float((acc_e != 0).sum().item()) / float(w.n_valid * w.H)
        del acc_e
        # algorithmic work: one pass of Q K^T over the domain (accumulate), 4*d per kept entry (forward);
        # the kernels recompute Q K^T once per sweep of the threshold iteration
        entmax = {"accumulate_ms": ent_ms[0], "sparse_fwd_ms": ent_ms[1],
                  "accumulate_one_pass_tflops": 2.0 * w.d * w.n_valid * w.H * w.B / (ent_ms[0] * 1e-3) / 1e12,
                  "fwd_effective_tflops": metrics.effective_flops(int(nnz.sum().item()), w.B, w.d) / (ent_ms[1] * 1e-3) / 1e12,
                  "entries_given_weight": support,
                  "note": "ap_accumulate_attention_entmax15 on one calibration batch into a scratch accumulator and "
                          "ap_sparse_attention_entmax15_fwd under the step's mask, %d runs after 2 warm-up runs; "
                          "entries_given_weight = fraction of the domain that received weight from any sample" % n_ent}

    # ---- the forward at other kept fractions on this shape, and the small workloads (outside the step) ----
    density = workloads = gathered = None
    if not args.no_extras:
        if w.dtype != "f32":
            density = density_section(ap, w, acc, q, k, v, out, ws, stage_ms["dense_fwd"], T_dense, peaks, dev)
            gathered = gathered_section(ap, w, acc, q, k, v, out, ws, dev)
        if world == 1:
            workloads = workloads_section(ap, dev, peaks, not args.no_cpu_baseline)

    # ---- the same step replayed from a CUDA graph (launch gaps of the ~25 kernels of a step removed) ----
    # (last: the replays add one calibration batch over and over, which skews the accumulator)
    graph_ms = None
    try:
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step(0)  # same stream as the capture: library state (function attributes) is set up
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(0)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        g0.record()
        for _ in range(args.steps):
            graph.replay()
        g1.record()
        barrier()
        graph_ms = g0.elapsed_time(g1) / args.steps
        (graph_ms,) = replicas.max_over_ranks(info, [graph_ms], dev)
        if ap.ap_device_status() != ap.AP_OK:
            raise RuntimeError("device status not OK after the graph replays")
    except RuntimeError as exc:  # capture refused: reported, not fatal
        graph_ms = "unavailable: %s" % str(exc).splitlines()[0][:120]

    if rank != 0:
        return
    # ---- rooflines ---------------------------------------------------------------------------------
    # The forward's algorithmic unit is the slot (128 query rows x 16 key columns): the kernel
    # executes exactly the slots of the schedule, 4*d*128*16 FLOPs each per batch element.  The
    # kept-tile figure (every stored 128x128 tile computed in full) is given beside it; it exceeds
    # what is executed because empty groups inside stored tiles are skipped.
    tile_fl = metrics.tile_flops(T_sparse, w.B, w.d)
    slot_fl = metrics.slot_flops(n_slots, w.B, w.d)
    fwd_s = stage_ms["sparse_fwd"] * 1e-3
    comp_bytes = metrics.compulsory_bytes(w.B, w.H, w.Lq, w.Lk, w.d, elem)
    tensor_bound = w.dtype == "bf16" and slot_fl / comp_bytes > peaks["bf16_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if tensor_bound:
        roof = {"bound": "tensor", "achieved": slot_fl / fwd_s / 1e12, "peak": peaks["bf16"],
                "unit": "TFLOP/s", "peak_kind": "bf16 burst (the forward is timed alone between events), of " + peaks["source"]}
    else:
        roof = {"bound": "hbm", "achieved": comp_bytes / fwd_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "peak_kind": "copy bandwidth, of " + peaks["source"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    traffic = NCU_TRAFFIC.get(w.name, {}) if (w.B, w.H) == (inputs.WORKLOADS[w.name].B, inputs.WORKLOADS[w.name].H) else {}
    roof["traffic"] = (traffic.get("sparse_fwd") or {}).get("bytes")
    roof["traffic_source"] = (traffic.get("sparse_fwd") or {}).get("source")
    roof["kernel"] = "sparse_fwd (fwd_tc_kernel)" if w.dtype == "bf16" else "sparse_fwd (fwd_simt_kernel)"
    roof["algorithmic"] = {"slot_flops": slot_fl, "slots_per_launch": n_slots * w.B, "rounds_per_launch": n_rounds * w.B,
                           "kept_tile_flops": tile_fl, "compulsory_bytes": comp_bytes, "tiles_per_step": T_sparse}
    roof["other_views"] = {"executed_flops_frac_of_bf16_sustained": slot_fl / fwd_s / 1e12 / peaks["bf16_sustained"],
                           "kept_tile_flops_frac_of_bf16_burst": tile_fl / fwd_s / 1e12 / peaks["bf16"],
                           "kept_tile_flops_frac_of_bf16_sustained": tile_fl / fwd_s / 1e12 / peaks["bf16_sustained"],
                           "effective_flops_frac_of_bf16_burst": eff_flops / fwd_s / 1e12 / peaks["bf16"],
                           "compulsory_bytes_frac_of_hbm": comp_bytes / fwd_s / 1e9 / peaks["hbm_gbs"]}
    # other stages, HBM view: accumulate = acc read+write over the domain + bias + Q,K;
    # build_mask = 2 reads of acc + mask bytes + bitmap bits over H*Lq*Lk
    dom = w.n_valid * w.H
    acc_bytes = 8.0 * dom + 4.0 * dom + elem * w.B * w.H * (w.Lq + w.Lk) * w.d
    mask_bytes = 8.0 * dom + 1.125 * w.H * w.Lq * w.Lk
    by_stage = {
        "accumulate": {"bound": "hbm", "achieved": acc_bytes / (stage_ms["accumulate"] * 1e-3) / 1e9,
                       "peak": peaks["hbm_gbs"], "unit": "GB/s"},
        "build_mask": {"bound": "hbm", "achieved": mask_bytes / (stage_ms["build_mask"] * 1e-3) / 1e9,
                       "peak": peaks["hbm_gbs"], "unit": "GB/s"},
        "dense_fwd": {"bound": "tensor", "unit": "TFLOP/s", "peak": peaks["bf16"],
                      "achieved": metrics.tile_flops(T_dense, w.B, w.d) / (stage_ms["dense_fwd"] * 1e-3) / 1e12},
    }
    for name, r in by_stage.items():
        r["frac"] = r["achieved"] / r["peak"]
        r["traffic"] = (traffic.get(name) or {}).get("bytes")
        r["traffic_source"] = (traffic.get(name) or {}).get("source")
    by_stage["dense_fwd"]["frac_of_bf16_sustained"] = by_stage["dense_fwd"]["achieved"] / peaks["bf16_sustained"]
    by_stage["accumulate"]["algorithmic_bytes"] = acc_bytes
    by_stage["build_mask"]["algorithmic_bytes"] = mask_bytes
    # the kernel with the largest share of the step's device time is not the metric's kernel
    share = {k: v / sum(stage_ms.values()) for k, v in stage_ms.items()}
    roof["step_share"] = share["sparse_fwd"]
    roof["largest_stage"] = {"stage": max(share, key=share.get), "share": max(share.values()),
                             "roofline": "roofline_by_stage"}

    # ---- CPU baseline (bounded sample) -----------------------------------------------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        units, seqs = min(w.H, 16), min(w.B, 4)
        r = oracle_sample_step(w, units, calib_seqs=seqs, batch=seqs)
        cpu = {"value": r["flops"] / r["fwd_s"] / 1e12, "unit": UNIT, "cores": r["cores"], "kind": "oracle",
               "sample": "forward of heads 0..%d of batch elements 0..%d (%d of %d (b,h) units), mask from %d "
                         "calibration sequences" % (units - 1, seqs - 1, units * seqs, w.B * w.H, seqs),
               "stage_seconds": {"accumulate": r["acc_s"], "build_mask": r["mask_s"], "sparse_fwd": r["fwd_s"]}}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": dict(workload_config(w),
                       l2="inputs exceed L2" if flush is None else "256 MiB flush write between steps",
                       value_scope="sparse forward's device time inside the step; ms_per_step is the whole step"),
        "stage_ms": stage_ms,
        "stage_ms_median": {s_: stage_all[s_]["median"] for s_ in stages},
        "stage_ms_best": {s_: stage_all[s_]["best"] for s_ in stages},
        "tokens_per_s": replicas.job_throughput(info, w.B * w.Lq, fwd_ms_max * 1e-3),
        "speedup_vs_dense_path": stage_ms["dense_fwd"] / stage_ms["sparse_fwd"],
        "mask": {"kept_fraction": nnz_total / float(dom), "tiles_kept": T_sparse, "tiles_domain": T_dense,
                    "tile_fill": nnz_total / (T_sparse * 128.0 * 128.0) if T_sparse else None},
        "pct_of_bf16_roofline": {"effective_flops_burst": 100 * eff_flops / fwd_s / 1e12 / peaks["bf16"],
                                 "tile_flops_burst": 100 * tile_fl / fwd_s / 1e12 / peaks["bf16"],
                                 "tile_flops_sustained": 100 * tile_fl / fwd_s / 1e12 / peaks["bf16_sustained"]},
        "pct_of_hbm_roofline": 100 * comp_bytes / fwd_s / 1e9 / peaks["hbm_gbs"],
        "roofline": roof, "roofline_by_stage": by_stage, "cpu_baseline": cpu,
        "e2e": {"value": replicas.job_throughput(info, eff_flops, e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches), "clocks": clocks, "layer_threshold": layer, "backward": backward,
        "entmax15": entmax, "workloads": workloads, "density": density, "gathered_rounds": gathered,
        "graph_replay": {"ms_per_step": graph_ms, "note": "the same step (same calibration batch every replay) "
                         "captured once in a CUDA graph; steps replays timed with one pair of events"},
    }
    print(json.dumps(line))


def run_density_sweep(args, w):
    """Speedup of the sparse forward over the library's dense path as a function of the kept
    fraction, on the workload's shape and calibration statistics (one GPU).  Two mask families:
    'topk' = the method's per-head top-fraction masks; 'blocks' = masks whose kept entries fill
    whole 128x128 tiles (the tiles with the largest accumulated mass), where tile occupancy tracks
    density.  Prints one JSON line with the table."""
    from paper_2012_02030_b200 import binding as ap

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    bias = inputs.calib_bias(w).to(dev)
    acc = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.float32, device=dev)
    for t in range(args.calib_batches if args.calib_batches > 0 else w.calib_batches):
        cq, ck = inputs.calib_qk(w, t)
        ap.ap_accumulate_attention(acc, cq.to(dev), ck.to(dev), bias, causal=w.causal)
    q, k, v = (t.to(dev) for t in inputs.eval_qkv(w))
    out = torch.empty_like(q)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    dense = ap.Tiles(w.H, w.Lq, w.Lk, device=dev)
    nnz = torch.zeros((w.H,), dtype=torch.int64, device=dev)
    ws = torch.empty(ap.ap_build_mask_workspace_bytes(w.H, w.Lq, w.Lk), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def time_fwd(tl):
        for _ in range(3):
            ap.ap_sparse_attention_fwd(q, k, v, tl, out)
        ms = []
        for _ in range(max(args.steps, 5)):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ap.ap_sparse_attention_fwd(q, k, v, tl, out)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        return float(np.median(ms))

    ap.ap_dense_tiles(dense, causal=w.causal)
    dense_ms = time_fwd(dense)
    n_qt, n_kt = dense.n_qt, dense.n_kt
    # accumulated mass per 128x128 tile, for the block-structured family
    pad_q, pad_k = n_qt * 128 - w.Lq, n_kt * 128 - w.Lk
    mass = torch.nn.functional.pad(acc, (0, pad_k, 0, pad_q)).view(w.H, n_qt, 128, n_kt, 128).sum((2, 4))
    dom_tiles = torch.ones((n_qt, n_kt), dtype=torch.bool, device=dev)
    if w.causal:
        dom_tiles = torch.tril(dom_tiles)
    rows = []
    for keep in (1.0, 0.5, 0.25, 0.1, 0.05, 0.02):
        ap.ap_build_mask(acc, keep, w.causal, w.keep_diag, None, tiles, nnz, ws)
        ms = time_fwd(tiles)
        n_rounds = int(tiles.round_ptr[-1].item())
        slots = int((tiles.round_info[:n_rounds] & 15).sum().item())
        rows.append({"family": "topk", "keep": keep, "kept_fraction": float(nnz.sum().item()) / (w.n_valid * w.H),
                     "tiles": tiles.n_tiles(), "slots": slots, "fwd_ms": ms, "speedup_vs_dense_path": dense_ms / ms,
                     "effective_tflops": metrics.effective_flops(int(nnz.sum().item()), w.B, w.d) / (ms * 1e-3) / 1e12})
    for keep in (1.0, 0.5, 0.25, 0.1, 0.05, 0.02):
        # keep the heaviest tiles of every head (the diagonal tiles always), entries inside the domain
        score = mass.masked_fill(~dom_tiles, float("-inf")).clone()
        idx = torch.arange(min(n_qt, n_kt), device=dev)
        score[:, idx, idx] = float("inf")
        n_keep = max(min(n_qt, n_kt), int(round(keep * int(dom_tiles.sum().item()))))
        thr = score.flatten(1).topk(n_keep, dim=1).values[:, -1]
        tile_keep = score >= thr[:, None, None]
        m = tile_keep[:, :, None, :, None].expand(w.H, n_qt, 128, n_kt, 128).reshape(w.H, n_qt * 128, n_kt * 128)
        m = m[:, :w.Lq, :w.Lk]
        if w.causal:
            m = m & torch.tril(torch.ones((w.Lq, w.Lk), dtype=torch.bool, device=dev))
        mask = m.to(torch.uint8).contiguous()
        ap.ap_mask_to_tiles(mask, tiles)
        kept = int(mask.sum().item())
        ms = time_fwd(tiles)
        n_rounds = int(tiles.round_ptr[-1].item())
        slots = int((tiles.round_info[:n_rounds] & 15).sum().item())
        rows.append({"family": "blocks", "keep": keep, "kept_fraction": kept / float(w.n_valid * w.H),
                     "tiles": tiles.n_tiles(), "slots": slots, "fwd_ms": ms, "speedup_vs_dense_path": dense_ms / ms,
                     "effective_tflops": metrics.effective_flops(kept, w.B, w.d) / (ms * 1e-3) / 1e12})
    if ap.ap_device_status() != ap.AP_OK:
        raise RuntimeError("device status not OK after the sweep")
    print(json.dumps({"density_sweep": {"workload": w.name, "dense_path_ms": dense_ms, "dense_tiles": dense.n_tiles(),
                                        "timing": "median of single launches, 256 MiB L2 flush before each",
                                        "rows": rows}}))


def main():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=10)
    p.add_argument("--warmup", type=int, default=3)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="long", choices=sorted(inputs.WORKLOADS))
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--calib-batches", type=int, default=0,
                   help="calibration batches accumulated before the timed steps (0 = the workload's own count); "
                        "profiling runs use a small number to keep the launch list short")
    p.add_argument("--B", type=int, default=0, help="override the workload's batch size (profiling runs use a small case)")
    p.add_argument("--H", type=int, default=0, help="override the workload's head count")
    p.add_argument("--no-extras", action="store_true",
                   help="leave out the sections measured outside the step (other densities, the small workloads)")
    p.add_argument("--density-sweep", action="store_true",
                   help="instead of the bench line: forward time vs kept fraction on the workload's shape")
    args = p.parse_args()
    w = inputs.WORKLOADS[args.workload]
    if args.B > 0 or args.H > 0:
        w = w.scaled(**({"B": args.B} if args.B > 0 else {}), **({"H": args.H} if args.H > 0 else {}))
    if args.density_sweep:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        run_density_sweep(args, w)
        return
    if args.impl == "reference":
        run_reference(args, w)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    run_gpu(args, w)
    replicas.shutdown(replicas.rank_info())


if __name__ == "__main__":
    main()
