#!/usr/bin/env python
"""Benchmark of the decode-fused GEMV path.

One "step" is one pass of the whole hot path over one batch of synthetic input: every matrix of the
workload's decoder layer, held Huffman-compressed in HBM, is multiplied with one bf16 activation
vector by the fused kernel (stream the compressed bytes, decode in registers, multiply, reduce).

    python bench.py --gpus 1 --steps 20 --warmup 5            # this library
    python bench.py --impl reference --steps 3 --warmup 1     # the CPU oracle on a bounded sample
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   # N independent replicas

Prints ONE JSON line (rank 0).  metric = uncompressed-equivalent weight GB/s (2 bytes per weight over
the step time); roofline = compressed bytes the kernels must read over their measured duration, against
the measured HBM copy bandwidth of this GPU pool.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "decode-fused GEMV uncompressed-equiv weight GB/s; % HBM roofline on comp. bytes"
UNIT = "GB/s"
WORKLOADS = {
    # name: (layer table, std, seed, description)
    "small_1024": ([("w", 1024, 1024)], 0.02, 1000, "single 1024x1024 bf16 matrix (oracle-sized case)"),
    "llama7b_layer": (wl.LAYER_LLAMA7B, 0.02, 2000, "Llama-7B-shaped decoder layer, 7 matrices, batch 1"),
    "8b_layer": (wl.LAYER_8B, 0.02, 3000, "8B-shaped decoder layer (GQA k/v 1024x4096, FFN 14336), batch 1"),
    "ffn70b": (wl.FFN_70B, 0.015, 4000, "70B-FFN-shaped pair 28672x8192 / 8192x28672"),
}
# Which matrices of a layer table may run in one launch.  "deps": only matrices that a decoder layer can really
# compute side by side (q,k,v read the same input; so do gate and up); "all": the whole table; "none": one each.
def launch_groups(table, fuse: str):
    n = len(table)
    if fuse == "none" or n == 1:
        return [[i] for i in range(n)]
    if fuse == "all":
        return [list(range(n))]
    names = [t[0] for t in table]
    if names[:7] == ["q", "k", "v", "o", "gate", "up", "down"]:
        return [[0, 1, 2], [3], [4, 5], [6]]
    return [[i] for i in range(n)]
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of the step's four fused-product launches over their algorithmic bytes, from the
# ncu capture summarised in profiles/huff_kernel_product_llama7b_layer.md (326.48 MB moved for 318.64 MB);
# traffic = ratio * algorithmic bytes.
NCU_TRAFFIC_RATIO = 1.025


def max_over_ranks(v: float, dist, device) -> float:
    """The slowest rank's time: replicas run independently, the job is as fast as its slowest member."""
    if dist is None:
        return v
    import torch
    t = torch.tensor([v], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(unc_bytes_per_rank: int, world: int, ms_step_max: float) -> float:
    """Uncompressed-equivalent GB/s of all replicas together (weak scaling: every rank does the whole workload)."""
    return world * unc_bytes_per_rank / (ms_step_max * 1e-3) / 1e9


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid, self.proc, self.lines = uuid, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def wait_first(self, limit_s: float):
        """Wait until the sampler has delivered its first line (or the limit has passed)."""
        t0 = time.time()
        while self.proc and not self.lines and time.time() - t0 < limit_s:
            time.sleep(0.02)

    def mark(self):
        """Only samples that arrive after this call count (if any do)."""
        self.first = len(self.lines)

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        first = getattr(self, "first", 0)
        for ln in (self.lines[first:] if len(self.lines) > first else self.lines):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def prepare(workload: str, chunk_elems: int, hl, torch, dev, cpu_sample_mats: int = 0, split: int = 0, batch: int = 1,
            wdtype: str = "bf16", max_code_len: int = 0):
    """Generate, encode (host) and upload every matrix of the workload."""
    table, std, seed, _ = WORKLOADS[workload]
    mats = []
    for i, (name, rows, cols) in enumerate(table):
        w = wl.gaussian_weights(rows, cols, std, seed + i, wdtype)
        cb = hl.build_codebook(w, hl.BF16 if wdtype == "bf16" else hl.FP16, max_code_len, split)
        blob, desc = hl.encode(cb, w, chunk_elems)
        cb.free()
        x = wl.activations(batch, cols, seed + 500 + i, "bf16" if wdtype == "bf16" else "fp16")
        ws_bytes = hl.workspace_bytes(desc, batch)
        alg_bytes = (desc.payload_bytes + 4 * (desc.n_chunks + 1) + (1 if wdtype == "bf16" else 3) * (4 << desc.lut_bits)
                     + batch * (2 * cols + 4 * rows))
        mats.append(dict(name=name, rows=rows, cols=cols, desc=desc, blob_dev=torch.from_numpy(blob).to(dev),
                         x_host=torch.from_numpy(x.view(np.int16).reshape(-1)).pin_memory(),
                         y_host=torch.zeros(batch * rows, dtype=torch.float32).pin_memory(),
                         x_dev=torch.from_numpy(x.view(np.int16).reshape(-1)).to(dev),
                         y_dev=torch.zeros(batch * rows, dtype=torch.float32, device=dev),
                         ws=torch.zeros(ws_bytes, dtype=torch.uint8, device=dev), ws_bytes=ws_bytes,
                         alg_bytes=int(alg_bytes), coded_bits=int(desc.coded_bits), raw_bits=int(desc.raw_bits),
                         blob_bytes=int(desc.blob_bytes), w_sample=w.copy() if i < cpu_sample_mats else None,
                         x_np=x[:1] if i < cpu_sample_mats else None))
        del w
    ws_each = max(m["ws_bytes"] for m in mats)       # a multi-matrix call states one size that every workspace must have
    for m in mats:
        m["ws"], m["ws_bytes"] = torch.zeros(ws_each, dtype=torch.uint8, device=dev), ws_each
    # activations and results of the whole step live in one host buffer and one device buffer each (the matrices'
    # tensors are views), so that a step's inputs go in with one copy and its results come out with one
    nx, ny = sum(m["x_dev"].numel() for m in mats), sum(m["y_dev"].numel() for m in mats)
    pk = dict(x_host=torch.empty(nx, dtype=torch.int16).pin_memory(), y_host=torch.zeros(ny, dtype=torch.float32).pin_memory(),
              x_dev=torch.empty(nx, dtype=torch.int16, device=dev), y_dev=torch.zeros(ny, dtype=torch.float32, device=dev))
    ox = oy = 0
    for m in mats:
        a, b = m["x_dev"].numel(), m["y_dev"].numel()
        pk["x_host"][ox:ox + a].copy_(m["x_host"])
        for key, buf, o, n in (("x_host", pk["x_host"], ox, a), ("x_dev", pk["x_dev"], ox, a), ("y_host", pk["y_host"], oy, b),
                               ("y_dev", pk["y_dev"], oy, b)):
            m[key] = buf[o:o + n]
        ox, oy = ox + a, oy + b
    pk["x_dev"].copy_(pk["x_host"])
    mats[0]["packed"] = pk
    return mats


def oracle_sample_time(hl, w_sample, x_np, chunk_elems: int, repeats: int = 1, fp16: bool = False):
    """Time the CPU oracle (bit-serial decode of the library's blob + fp64 product) on a sample tensor."""
    from oracle import oracle as orc
    cb = hl.build_codebook(w_sample, hl.FP16 if fp16 else hl.BF16)
    blob, _ = hl.encode(cb, w_sample, chunk_elems)
    cb.free()
    orc.lib()
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        back, _ = orc.decode_blob(blob)
        y, _ = orc.matmul(back, x_np, orc.FP16 if fp16 else orc.BF16)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    assert np.array_equal(back, w_sample)
    return best


def _oracle_one(item):
    """Worker of the all-cores leg: the oracle's decode of one blob and its fp64 product (runs in a forked child)."""
    from oracle import oracle as orc
    blob, w, x, fp16 = item
    back, _ = orc.decode_blob(blob)
    orc.matmul(back, x, orc.FP16 if fp16 else orc.BF16)
    return bool(np.array_equal(back, w))


def oracle_parallel_time(hl, parts, chunk_elems: int, procs: int, fp16: bool = False):
    """The same oracle calls on several tensors at once, one host process per core (forked from the harness, which hands
    each child its tensors; the oracle itself stays single-threaded and untouched): wall time of the whole batch."""
    import multiprocessing as mp
    from concurrent.futures import ProcessPoolExecutor
    from oracle import oracle as orc
    orc.lib()
    items = []
    for w, x in parts:
        cb = hl.build_codebook(w, hl.FP16 if fp16 else hl.BF16)
        blob, _ = hl.encode(cb, w, chunk_elems)
        cb.free()
        items.append((blob, w, x, fp16))
    global _FORK_ITEMS
    _FORK_ITEMS = items                      # children inherit the tensors through fork: nothing is pickled on the way in
    with ProcessPoolExecutor(max_workers=procs, mp_context=mp.get_context("fork")) as ex:
        list(ex.map(_fork_warm, range(procs)))             # children are up (and have loaded the oracle) before the clock starts
        t0 = time.perf_counter()
        ok = list(ex.map(_fork_run, range(len(items))))
        dt = time.perf_counter() - t0
    _FORK_ITEMS = None
    assert all(ok)
    return dt


_FORK_ITEMS = None


def _fork_warm(_):
    from oracle import oracle as orc
    orc.lib()
    return True


def _fork_run(i):
    return _oracle_one(_FORK_ITEMS[i])


def row_parts(w, x, n_parts: int):
    """Cut a matrix into up to n_parts blocks of whole 16-row tiles."""
    rows = w.shape[0]
    per = max(16, (rows + n_parts - 1) // n_parts // 16 * 16)
    return [(w[r:r + per].copy(), x) for r in range(0, rows, per)]


def run_reference(args):
    """The oracle arm: the CPU oracle, as it stands, on a bounded sample of the same workload (one host thread)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import paper_2502_00922_b200 as hl   # host encoder only: it produces the blob the oracle decodes
    table, std, seed, desc_text = WORKLOADS[args.workload]
    total_rows = sum(r for _, r, _ in table)
    total_weights = sum(r * c for _, r, c in table)
    # probe: 16 rows of the first matrix; then size the per-step sample so that warm-up + K steps take about 90 s,
    # the same share of the rows of every matrix of the step (16-row granularity, at least one tile each)
    name0, rows0, cols0 = table[0]
    w0 = wl.gaussian_weights(64, cols0, std, seed)
    x0 = wl.activations(1, cols0, seed + 500)
    probe = oracle_sample_time(hl, w0, x0, args.chunk_elems) / w0.size           # seconds per weight
    budget_weights = 90.0 / (probe * (args.warmup + args.steps))
    share = min(1.0, budget_weights / total_weights)
    sample = []
    for i, (name, rows, cols) in enumerate(table):
        n = int(max(16, min(rows, int(rows * share) // 16 * 16)))
        sample.append((wl.gaussian_weights(rows, cols, std, seed + i)[:n].copy(), wl.activations(1, cols, seed + 500 + i)))
    n_w = sum(w.size for w, _ in sample)
    times = []
    for i in range(args.warmup + args.steps):
        dt = sum(oracle_sample_time(hl, w, x, args.chunk_elems) for w, x in sample)
        if i >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    value = 2.0 * n_w / t / 1e9
    text = (f"per step the first {100.0 * n_w / total_weights:.3f} % of the rows of each of the {len(table)} matrices "
            f"({n_w} weights): bit-serial decode of the blobs + fp64 products, one thread")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": {"workload": args.workload, "what": desc_text, "sample": text},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": text},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def small_batch_leg(hl, torch, dev, stream, chunk_elems: int, peak_for_small: float):
    """One 70B-FFN-shaped matrix (28672 x 8192) at batch 1, 16, 32 and 64: ms per product, fraction of the HBM peak on the
    compressed bytes, and which kernel ran."""
    name, rows, cols = wl.FFN_70B[0]
    w = wl.gaussian_weights(rows, cols, 0.015, 4000)
    cb = hl.build_codebook(w)
    blob, desc = hl.encode(cb, w, chunk_elems)
    cb.free()
    del w
    blob_dev = torch.from_numpy(blob).to(dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_bytes = hl.workspace_bytes(desc, 64)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    out = {"matrix": f"{rows}x{cols}", "chunk_elems": chunk_elems, "compressed_bytes": int(desc.blob_bytes), "batches": []}
    for batch in (1, 16, 32, 64):
        x = torch.from_numpy(wl.activations(batch, cols, 4500 + batch).view(np.int16).reshape(-1)).to(dev)
        y = torch.zeros(batch * rows, dtype=torch.float32, device=dev)
        for _ in range(5):
            hl.decode_gemm(desc, blob_dev, x, batch, y, ws, ws_bytes, err, stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        n = 200
        a.record(stream)
        for _ in range(n):
            hl.decode_gemm(desc, blob_dev, x, batch, y, ws, ws_bytes, err, stream)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / n
        alg = desc.payload_bytes + 4 * (desc.n_chunks + 1) + (4 << desc.lut_bits) + batch * (2 * cols + 4 * rows)
        out["batches"].append({"batch": batch, "ms": ms, "frac_of_hbm_peak": alg / (ms * 1e-3) / 1e9 / peak_for_small,
                               "uncompressed_GBs": 2.0 * rows * cols / (ms * 1e-3) / 1e9,
                               "kernel": "huff_kernel<product, one vector> (mixed-precision fma on the decoded registers)" if batch == 1 else
                                         "huff_kernel<product> (mma.sync on the decoded registers)" if batch <= 8 else
                                         ("huff_kernel<product, two tiles of activations> (mma.sync on the decoded registers)" if batch <= 16
                                          else "huff_gemm_tc_kernel (tcgen05)")})
    assert int(err.item()) == 0
    return out


def fp16_leg(hl, torch, dev, stream, chunk_elems: int, peak: float):
    """The paper's FP16 {1,5,5,5} format (Section 3.1) on one matrix of the layer (gate, 11008 x 4096) with fp16-trained
    weights, batch 1, at the benchmark's chunk size: ms per product and fraction of the HBM peak on the compressed bytes."""
    name, rows, cols = "gate", 11008, 4096
    w = wl.gaussian_weights(rows, cols, 0.02, 1000 + 4, "fp16")
    cb = hl.build_codebook(w, hl.FP16)
    blob, desc = hl.encode(cb, w, chunk_elems)
    cb.free()
    del w
    blob_dev = torch.from_numpy(blob).to(dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_bytes = hl.workspace_bytes(desc, 1)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    x = torch.from_numpy(wl.activations(1, cols, 1504, "fp16").view(np.int16).reshape(-1)).to(dev)
    y = torch.zeros(rows, dtype=torch.float32, device=dev)
    for _ in range(5):
        hl.decode_gemv(desc, blob_dev, x, y, ws, ws_bytes, err, stream)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    n = 400
    a.record(stream)
    for _ in range(n):
        hl.decode_gemv(desc, blob_dev, x, y, ws, ws_bytes, err, stream)
    b.record(stream)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ms = a.elapsed_time(b) / n
    alg = desc.payload_bytes + 4 * (desc.n_chunks + 1) + 3 * (4 << desc.lut_bits) + 2 * cols + 4 * rows
    plan = hl.decode_launch_plan(desc, 1)
    return {"matrix": f"{name} {rows}x{cols}", "weights": "fp16-trained (gaussian), FP16 {1,5,5,5}", "chunk_elems": chunk_elems,
            "compressed_bytes": int(desc.blob_bytes), "compression_ratio_total": 2.0 * rows * cols / desc.blob_bytes,
            "ms": ms, "frac_of_hbm_peak": alg / (ms * 1e-3) / 1e9 / peak, "uncompressed_GBs": 2.0 * rows * cols / (ms * 1e-3) / 1e9,
            "flat_fields": int(desc.flat_fields), "slots_per_warp": plan["slots_per_warp"], "decoder_warps": plan["decoder_warps"],
            "kernel": "huff_kernel<product, one vector, FP16" + (", flat mantissa codes>" if desc.flat_fields & 6 == 6 else ">")}


def sweep_8b_leg(hl, torch, dev, stream, chunk_elems: int, peak: float, layers: int = 32):
    """The per-token pass over an 8B-shaped model: `layers` decoder layers, every layer with its own copy of the seven
    blobs in HBM (same content, distinct memory), four launches per layer, batch 1; beside it the dense bf16 sweep of the
    same shapes in the same launch groups."""
    mats = prepare("8b_layer", chunk_elems, hl, torch, dev)
    table = WORKLOADS["8b_layer"][0]
    groups = launch_groups(table, "deps")
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_each = max(m["ws_bytes"] for m in mats)
    blobs = [[m["blob_dev"] for m in mats]] + [[m["blob_dev"].clone() for m in mats] for _ in range(layers - 1)]
    preps = [hl.PreparedMulti([mats[i]["desc"] for i in g], [bl[i] for i in g], [mats[i]["x_dev"] for i in g], 1,
                              [mats[i]["y_dev"] for i in g], [mats[i]["ws"] for i in g], ws_each, err) for bl in blobs for g in groups]
    raw = stream.cuda_stream

    def timed(fn, n):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    ms = timed(lambda: [p.run(raw) for p in preps], 30)
    assert int(err.item()) == 0
    n_w = layers * sum(r * c for _, r, c in table)
    alg = layers * sum(m["alg_bytes"] for m in mats)
    out = {"workload": f"8B-shaped model, {layers} layers, batch 1, {len(preps)} launches per token", "weights": n_w,
           "compressed_bytes_resident": layers * sum(m["blob_bytes"] for m in mats), "ms_per_token": ms, "ms_per_layer": ms / layers,
           "tokens_per_s_equiv": 1e3 / ms, "uncompressed_GBs": 2.0 * n_w / (ms * 1e-3) / 1e9,
           "frac_of_hbm_peak_on_compressed_bytes": alg / (ms * 1e-3) / 1e9 / peak}
    del preps, blobs
    try:
        dense = [[torch.empty((r, c), dtype=torch.int16, device=dev) for _, r, c in table] for _ in range(layers)]
        for lw in dense:
            for w_dev in lw:
                w_dev.view(torch.bfloat16).normal_(0, 0.02)
        dpreps = [hl.PreparedPlainMulti([lw[i] for i in g], [table[i][1] for i in g], [table[i][2] for i in g],
                                        [mats[i]["x_dev"] for i in g], [mats[i]["y_dev"] for i in g]) for lw in dense for g in groups]
        dms = timed(lambda: [p.run(raw) for p in dpreps], 30)
        out["dense_bf16_ms_per_token"] = dms
        out["speedup_vs_dense"] = dms / ms
        del dense, dpreps
    except Exception as ex:
        print(f"[bench] dense sweep skipped: {ex}", file=sys.stderr)
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_layer", choices=sorted(WORKLOADS))
    ap.add_argument("--chunk-elems", type=int, default=4096)
    ap.add_argument("--fuse", default="deps", choices=["none", "deps", "all"],
                    help="which matrices of the layer share a launch")
    ap.add_argument("--split", default="paper", choices=["paper", "whole-exponent"],
                    help="field split of the blobs: the paper's BF16 {1,4,4,7} or {1,8,7} (one 256-symbol exponent code)")
    ap.add_argument("--max-code-len", type=int, default=0, help="L_max of the codebooks (0 = the library's default, 8; range 8..12, Section 3.2 quotes 12; above 9 the kernels look long codewords up in two levels)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16", "fp16_from_bf16"],
                    help="weight format: bf16 {1,4,4,7} blobs, or fp16 {1,5,5,5} blobs of true fp16 weights / of bf16 weights "
                         "stored as fp16 (use --chunk-elems 1024 for fp16: larger records do not fit 32 warps' slots)")
    ap.add_argument("--batch", type=int, default=1,
                    help="activation vectors per product (1..64; above 8 every matrix is its own launch: 9..16 on the register "
                         "path with two tiles of activations, above that on the tcgen05 path)")
    ap.add_argument("--layers", type=int, default=1,
                    help="sweep through this many decoder layers per step (each layer has its own copy of the blobs in HBM): "
                         "the per-token pass over a whole model, e.g. --workload 8b_layer --layers 32")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-small-batch", action="store_true",
                    help="skip the extra leg that times one 70B-FFN-shaped matrix at batch 1 / 16 / 64")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the extra leg that sweeps 32 layers of the 8B-shaped model (11 GB of blobs resident)")
    ap.add_argument("--repeats", type=int, default=0,
                    help="timed regions of exactly --steps steps each (0: as many as fill about 0.8 s, so that the clock "
                         "sampler sees the GPU under load); the line's ms_per_step is the median region, min and max are reported")
    ap.add_argument("--explore-splits", action="store_true",
                    help="also count and report the entropy of other bit-field splits of the workload's largest matrix (Section 3.1 table)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2502_00922_b200 as hl
    hl.lib()   # fails loudly when the CUDA library has not been built
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    args.warmup = max(args.warmup, 3)

    cpu_mats = 0 if (args.no_cpu_baseline or world > 1 or rank != 0) else 7      # whole matrices kept for the CPU-oracle leg (about 20 s)
    split = 0 if args.split == "paper" else 1
    B = args.batch
    if not 1 <= B <= 64:
        raise SystemExit("--batch must be in [1, 64]")
    fp16 = args.dtype != "bf16"
    # launches over several matrices take up to 8 vectors, up to 16 for BF16 blobs with 8-bit tables (two tiles of activations),
    # and 17 to 64 on the tensor-core kernel for tables of up to 9 bits (FP16: 8)
    multi = (B <= 8 or (B <= 16 and not fp16 and args.max_code_len in (0, 8))
             or (B > 16 and args.max_code_len in ((0, 8) if fp16 else (0, 8, 9))))
    if not multi:
        args.fuse = "none"           # one matrix per launch (passes of 8 vectors, or the tensor-core kernel at 9..16)
    mats = prepare(args.workload, args.chunk_elems, hl, torch, dev, cpu_mats, split, B, args.dtype, args.max_code_len)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    L = args.layers
    if L < 1 or (L > 1 and not multi):
        raise SystemExit("--layers must be at least 1 (and takes --batch up to 8)")
    n_weights = L * sum(m["rows"] * m["cols"] for m in mats)
    unc_bytes = 2 * n_weights
    alg_bytes = L * sum(m["alg_bytes"] for m in mats)
    stream = torch.cuda.current_stream()

    # every layer of the sweep streams its own copy of the blobs from HBM (same content, distinct memory)
    layer_blobs = [[m["blob_dev"] for m in mats]] + [[m["blob_dev"].clone() for m in mats] for _ in range(L - 1)]
    groups = launch_groups(WORKLOADS[args.workload][0], args.fuse)
    calls = [dict(descs=[mats[i]["desc"] for i in g], blobs=[blobs[i] for i in g], xs=[mats[i]["x_dev"] for i in g],
                  ys=[mats[i]["y_dev"] for i in g], wss=[mats[i]["ws"] for i in g]) for blobs in layer_blobs for g in groups]
    groups = groups * L              # one entry per launch of the step

    ws_each = max(m["ws_bytes"] for m in mats)
    raw_stream = stream.cuda_stream
    for c, g in zip(calls, groups):      # argument arrays marshalled once per launch group
        c["prep"] = hl.PreparedMulti(c["descs"], c["blobs"], c["xs"], B if multi else 8, c["ys"], c["wss"], ws_each, err,
                                     [mats[i]["x_host"] for i in g], [mats[i]["y_host"] for i in g])

    def step_device():
        if not multi:
            for m in mats:
                hl.decode_gemm(m["desc"], m["blob_dev"], m["x_dev"], B, m["y_dev"], m["ws"], m["ws_bytes"], err, stream)
            return
        for c in calls:
            c["prep"].run(raw_stream)

    for c, g in zip(calls, groups):
        c["xh"], c["yh"] = [mats[i]["x_host"] for i in g], [mats[i]["y_host"] for i in g]

    def step_host():      # host activations in, host results out
        if not multi:
            # activations staged by a copy kernel, results written to pinned host memory by the kernels, one wait per step
            for m in mats:
                hl.stage_copy(m["x_dev"], m["x_host"], m["x_host"].numel() * 2, stream)
                hl.decode_gemm(m["desc"], m["blob_dev"], m["x_dev"], B, m["y_host"], m["ws"], m["ws_bytes"], err, stream)
            stream.synchronize()
            return
        # the step's activations in with one copy from pinned memory, the launches, the step's results out with one copy
        pk = mats[0]["packed"]
        pk["x_dev"].copy_(pk["x_host"], non_blocking=True)
        for c in calls:
            c["prep"].run(raw_stream)
        pk["y_host"].copy_(pk["y_dev"], non_blocking=True)
        stream.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: R regions of exactly K steps each, every region between its own pair of events on the
    # launching stream, all regions back to back (no host wait in between) so that the GPU stays under load
    for _ in range(args.warmup):
        step_device()
    uuid = str(getattr(torch.cuda.get_device_properties(dev), "uuid", local))
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") or uuid.isdigit() else "GPU-" + uuid)
    barrier()
    probe_a, probe_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    probe_a.record(stream)
    for _ in range(args.steps):
        step_device()
    probe_b.record(stream)
    barrier()
    est_ms = max(probe_a.elapsed_time(probe_b), 1e-3)                  # one region, untimed: sizes the number of regions
    R = args.repeats if args.repeats > 0 else int(min(2000, max(5, 800.0 / est_ms)))
    sampler.start()
    sampler.wait_first(3.0)               # let the sampler come up before the timed regions start
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(R + 1)]
    barrier()
    sampler.mark()                        # samples from here on were taken under load
    evs[0].record(stream)
    for r in range(R):
        for s_ in range(args.steps):
            step_device()
        evs[r + 1].record(stream)
    barrier()
    clocks = sampler.stop()
    region_ms = [evs[r].elapsed_time(evs[r + 1]) / args.steps for r in range(R)]
    ms_step = max_over_ranks(statistics.median(region_ms), dist, dev)
    ms_min, ms_max = max_over_ranks(min(region_ms), dist, dev), max_over_ranks(max(region_ms), dist, dev)
    assert int(err.item()) == 0, "device error flag set"

    # ---- per-matrix durations (a second, shorter pass with an event after every launch)
    n_b = min(args.steps, 50)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(mats) + 1)] for _ in range(n_b)]
    for s in range(n_b):
        ev[s][0].record(stream)
        for i, m in enumerate(mats):
            hl.decode_gemm(m["desc"], m["blob_dev"], m["x_dev"], B, m["y_dev"], m["ws"], m["ws_bytes"], err, stream)
            ev[s][i + 1].record(stream)
    barrier()
    per_mat_ms = [statistics.median(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(n_b)) for i in range(len(mats))]
    kernel_ms_step = ms_step              # launches run back to back: average launch duration = step time / launches

    # ---- the same step as ONE launch over all matrices (valid where the products are independent, as they are here; a
    # decoder layer's data dependencies allow only the default grouping): reported beside the headline, not as it
    one_launch_ms = None
    if L == 1 and multi and len(mats) > 1 and len(groups) > 1 and len(mats) <= 8:
        allp = hl.PreparedMulti([m["desc"] for m in mats], [m["blob_dev"] for m in mats], [m["x_dev"] for m in mats], B,
                                [m["y_dev"] for m in mats], [m["ws"] for m in mats], ws_each, err)
        for _ in range(args.warmup):
            allp.run(raw_stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record(stream)
        for _ in range(args.steps):
            allp.run(raw_stream)
        b.record(stream)
        barrier()
        one_launch_ms = max_over_ranks(a.elapsed_time(b) / args.steps, dist, dev)

    # ---- plain decompression of the same blobs to 16-bit weights (huffllm_decode): reads the blobs, writes 2 bytes per weight
    decode_ms = None
    if rank == 0 and L == 1:
        big = max(mats, key=lambda m: m["rows"] * m["cols"])
        out_dev = torch.empty(big["rows"] * big["cols"], dtype=torch.int16, device=dev)
        n_d = min(args.steps, 100)
        for it in range(3 + n_d):
            if it == 3:
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
            for m in mats:
                hl.decode(m["desc"], m["blob_dev"], out_dev, err, stream)
        b.record(stream)
        torch.cuda.synchronize()
        decode_ms = a.elapsed_time(b) / n_d
        del out_dev

    # ---- end to end: x from pinned host memory, y back to the host, every step.  The step (copy in, launches, copy out)
    # is captured once in a CUDA graph where that works — the library's calls only enqueue work on the stream they are
    # given — and replayed with one wait per step; otherwise the calls are issued one by one.
    for _ in range(args.warmup):
        step_host()
    barrier()
    e2e_mode = "stream" if multi else ("stream; activations staged from pinned host memory by a copy kernel, results written to pinned "
                                         "host memory by the product kernels, one wait per step")
    run_e2e = step_host
    if multi:
        try:
            gstream = torch.cuda.Stream(device=dev)
            graph = torch.cuda.CUDAGraph()
            pk = mats[0]["packed"]
            # Inside a graph a DMA copy node between kernel nodes costs about 10 us, so the step moves its data with
            # kernels: the activations are staged from pinned host memory by huffllm_stage_copy, and the launches of the
            # (last) layer get the pinned host buffers as their y, so the results are written to the host as they are produced.
            n_last = len(calls) // L
            for c, g in zip(calls[-n_last:], groups[-n_last:]):
                c["prep_host_y"] = hl.PreparedMulti(c["descs"], c["blobs"], c["xs"], B if multi else 8, [mats[i]["y_host"] for i in g],
                                                    c["wss"], ws_each, err)
            x_bytes = pk["x_host"].numel() * pk["x_host"].element_size()
            assert x_bytes % 16 == 0
            with torch.cuda.stream(gstream):
                gstream.wait_stream(stream)
                with torch.cuda.graph(graph, stream=gstream):
                    hl.stage_copy(pk["x_dev"], pk["x_host"], x_bytes, gstream.cuda_stream)
                    for c in calls:
                        c.get("prep_host_y", c["prep"]).run(gstream.cuda_stream)
            def run_graph():
                graph.replay()               # on the current stream
                stream.synchronize()
            y_want = pk["y_dev"].cpu()       # from the device-resident steps above: same inputs, same sums
            pk["y_host"].fill_(float("nan"))
            run_graph()
            assert bool(torch.equal(pk["y_host"], y_want)), "graph replay did not deliver the step's results"
            run_e2e, e2e_mode = run_graph, ("cuda graph; activations staged from pinned host memory by a copy kernel, results written to "
                                            "pinned host memory by the product kernels, one wait per step")
        except Exception as ex:          # capture is an optimisation of the harness, never a requirement
            print(f"[bench] CUDA graph capture of the step skipped: {ex}", file=sys.stderr)
            torch.cuda.synchronize()
    for _ in range(args.warmup):
        run_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run_e2e()
    barrier()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / args.steps, dist, dev)

    # ---- the dense product the compression competes with: same layer, uncompressed bf16, own kernel and cuBLAS
    plain_ms = cublas_ms = None
    if rank == 0 and not fp16:
        try:
            dense = [(torch.randint(-2**15, 2**15, (m["rows"], m["cols"]), dtype=torch.int16, device=dev), m) for _ in range(L) for m in mats]
            for w_dev, m in dense:
                w_dev.view(torch.bfloat16).normal_(0, 0.02)
            # the dense layer in the same launch groups as the compressed one
            n_g = len(groups) // L
            dense_preps = [hl.PreparedPlainMulti([dense[l * len(mats) + i][0] for i in g], [mats[i]["rows"] for i in g],
                                                 [mats[i]["cols"] for i in g], [mats[i]["x_dev"] for i in g],
                                                 [mats[i]["y_dev"] for i in g]) for l in range(L) for g in groups[:n_g]]
            def plain():
                for p in dense_preps:
                    p.run(raw_stream)
            def cublas():
                for w_dev, m in dense:
                    torch.mv(w_dev.view(torch.bfloat16), m["x_dev"][:m["cols"]].view(torch.bfloat16))
            for fn, key in ((plain, "plain"), (cublas, "cublas")):
                for _ in range(args.warmup):
                    fn()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a.record(stream)
                for _ in range(args.steps):
                    fn()
                b.record(stream)
                torch.cuda.synchronize()
                if key == "plain":
                    plain_ms = a.elapsed_time(b) / args.steps
                else:
                    cublas_ms = a.elapsed_time(b) / args.steps
            del dense
        except Exception as ex:   # the comparison point must never take the benchmark down
            print(f"[bench] dense comparison skipped: {ex}", file=sys.stderr)

    # ---- the entropy table of Section 3.1 on the workload's largest matrix: device counting pass + host entropies
    explorer = None
    if rank == 0 and args.explore_splits:
        table, std, seed, _ = WORKLOADS[args.workload]
        i_big = max(range(len(table)), key=lambda i: table[i][1] * table[i][2])
        name, rows, cols = table[i_big]
        w_dev = torch.from_numpy(wl.gaussian_weights(rows, cols, std, seed + i_big, args.dtype).view(np.int16)).to(dev)
        splits = [[16], [8, 8], [1, 5, 5, 5], [4, 4, 4, 4]] if fp16 else [[16], [8, 8], [1, 8, 7], [1, 4, 4, 7]]
        explorer = {"matrix": name, "weights": rows * cols, "rows": []}
        for widths in splits:
            counts = torch.zeros(hl.split_counts_size(widths), dtype=torch.int64, device=dev)
            for _ in range(3):
                hl.split_histogram(w_dev, rows * cols, widths, counts, stream)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(20):
                hl.split_histogram(w_dev, rows * cols, widths, counts, stream)
            b.record(stream)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / 20
            ent, huf = hl.split_entropy(counts.cpu().numpy().view(np.uint64), widths)
            explorer["rows"].append({"split": "-".join(map(str, widths)), "entropy_bits": [round(float(x), 4) for x in ent],
                                     "total_bits_per_param": round(float(ent.sum()), 4), "huffman_bits_per_param": round(float(huf.sum()), 4),
                                     "ms": ms, "GBs_read": 2 * rows * cols * (2 if widths == [16] else 1) / (ms * 1e-3) / 1e9})
        # compression of that matrix where it sits: counts (above), codebook from the counts, encoder on the device
        hd = hl.FP16 if fp16 else hl.BF16
        widths = [1, 5, 5, 5] if fp16 else [1, 8, 7]
        counts = torch.zeros(hl.split_counts_size(widths), dtype=torch.int64, device=dev)
        cap = hl.encode_bound(rows, cols, hd, args.chunk_elems)
        blob_dev = torch.zeros(cap, dtype=torch.uint8, device=dev)
        n_scr = hl.encode_device_scratch_bytes(rows, cols, args.chunk_elems)
        scr = torch.zeros(n_scr, dtype=torch.uint8, device=dev)
        def compress():
            hl.split_histogram(w_dev, rows * cols, widths, counts, stream)
            c = counts.cpu().numpy().view(np.uint64)
            cb = hl.build_codebook_from_counts(c[2:98] if fp16 else c[2:258], hd, args.max_code_len, split)
            d = hl.encode_device(cb, w_dev, rows, cols, args.chunk_elems, blob_dev, cap, scr, n_scr, stream)
            cb.free()
            return d
        compress()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(5):
            d_enc = compress()
        torch.cuda.synchronize()
        dev_ms = (time.perf_counter() - t0) * 1e3 / 5
        w_host = w_dev.cpu().numpy().view(np.uint16)
        t0 = time.perf_counter()
        cb = hl.build_codebook(w_host, hd, args.max_code_len, split)
        blob_h, _ = hl.encode(cb, w_host, args.chunk_elems)
        host_ms = (time.perf_counter() - t0) * 1e3
        cb.free()
        explorer["compress"] = {"device_ms": dev_ms, "host_ms": host_ms, "same_blob": bool(np.array_equal(blob_dev[:d_enc.blob_bytes].cpu().numpy(), blob_h)),
                                "device_GBs_of_weights": 2 * rows * cols / (dev_ms * 1e-3) / 1e9,
                                "note": "counting pass + codebook from the counts + device encoder, wall clock including its two waits; host: codebook + encoder on the host cores"}
        del w_dev, blob_dev

    # ---- the CPU oracle on a bounded sample of the same workload (rank 0, single GPU run only): one thread, and the
    # same calls chunk-parallel over all host cores (the harness cuts the matrices into row blocks; the oracle is untouched)
    cpu = cpu_all = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = [m for m in mats if m["w_sample"] is not None]
        dt = sum(oracle_sample_time(hl, m["w_sample"], m["x_np"], args.chunk_elems, repeats=1, fp16=fp16) for m in sample)
        n_w = sum(m["w_sample"].size for m in sample)
        cpu = {"value": 2.0 * n_w / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"matrices {[m['name'] for m in sample]} in full ({n_w} weights = {100.0 * n_w / n_weights * L:.0f} % of a layer, "
                         f"{dt:.1f} s): bit-serial decode of the blob + fp64 product, one thread"}
        cores = os.cpu_count() or 1
        parts = [p for m in sample for p in row_parts(m["w_sample"], m["x_np"], 4 * cores)]
        dt_all = oracle_parallel_time(hl, parts, args.chunk_elems, cores, fp16)
        cpu_all = {"value": 2.0 * n_w / dt_all / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"the same {n_w} weights cut into {len(parts)} row blocks, {cores} host processes ({dt_all:.1f} s)"}

    # ---- one 70B-FFN-shaped matrix at batch 1 / 16 / 64: register path and tensor-core path under the same clock
    small_batch = None
    fp16_one = None
    if rank == 0 and world == 1 and not args.no_small_batch and not fp16 and args.workload == "llama7b_layer" and L == 1:
        small_batch = small_batch_leg(hl, torch, dev, stream, args.chunk_elems, peak_for_small=measured_peak()[0])
        fp16_one = fp16_leg(hl, torch, dev, stream, args.chunk_elems, measured_peak()[0])
    sweep_8b = None
    if rank == 0 and world == 1 and not args.no_sweep and not fp16 and args.workload == "llama7b_layer" and L == 1 and B == 1:
        sweep_8b = sweep_8b_leg(hl, torch, dev, stream, args.chunk_elems, measured_peak()[0])

    if rank != 0:
        return
    peak, peak_src = measured_peak()
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    value = whole_job_value(unc_bytes, world, ms_step)
    achieved = alg_bytes / (kernel_ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp16" if fp16 else "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "what": WORKLOADS[args.workload][3], "chunk_elems": args.chunk_elems, "batch": B, "layers": L,
                   "split": ("fp16 {1,5,5,5}" + (" of bf16-origin weights" if args.dtype == "fp16_from_bf16" else "")) if fp16 else
                            ("bf16 {1,4,4,7}" if args.split == "paper" else "bf16 {1,8,7} (whole exponent)"),
                   "max_code_len": int(mats[0]["desc"].lut_bits), "weights_per_step": n_weights,
                   "uncompressed_bytes": unc_bytes, "compressed_bytes": L * sum(m["blob_bytes"] for m in mats),
                   "compression_ratio_total": unc_bytes / (L * sum(m["blob_bytes"] for m in mats)),
                   "compression_ratio_payload": 16.0 * n_weights / (L * sum(m["coded_bits"] + m["raw_bits"] for m in mats)),
                   "bits_per_param_payload": L * sum(m["coded_bits"] + m["raw_bits"] for m in mats) / n_weights,
                   "l2": "inputs larger than L2: the step streams %.0f MB of compressed weights, L2 is 126 MB" % (alg_bytes / 1e6),
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "launch_groups": [[mats[i]["name"] for i in g] for g in groups[:len(groups) // L]],
                   "ms_per_layer": ms_step / L, "tokens_per_s_equiv": 1e3 / ms_step},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None if NCU_TRAFFIC_RATIO is None else NCU_TRAFFIC_RATIO * alg_bytes / len(groups),
                     "traffic_per_step": None if NCU_TRAFFIC_RATIO is None else NCU_TRAFFIC_RATIO * alg_bytes,
                     "traffic_note": "DRAM bytes read + written per launch (average over the step's launches): algorithmic bytes x the "
                                     "ratio of the ncu capture in profiles/ (1.025)",
                     "peak_source": peak_src, "kernel": "huff_kernel<product>" if B <= 8 else ("huff_kernel<product, two tiles>" if multi and B <= 16 else "huff_gemm_tc_kernel"), "launches_per_step": len(groups), "fuse": args.fuse,
                     "algorithmic_bytes_per_step": alg_bytes, "kernel_ms_per_step": kernel_ms_step,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "one_launch": None if not one_launch_ms else {
                         "ms_per_step": one_launch_ms, "value": whole_job_value(unc_bytes, world, one_launch_ms),
                         "frac": alg_bytes / (one_launch_ms * 1e-3) / 1e9 / peak,
                         "note": "all matrices of the step in one launch: only valid where their inputs are independent"},
                     "per_matrix": [{"name": m["name"], "rows": m["rows"], "cols": m["cols"], "ms": t,
                                     "comp_GBs": m["alg_bytes"] / (t * 1e-3) / 1e9} for m, t in zip(mats, per_mat_ms)]},
        "cpu_baseline": cpu,
        "e2e": {"value": whole_job_value(unc_bytes, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms, "submission": e2e_mode,
                "h2d_bytes_per_step": B * sum(2 * m["cols"] for m in mats), "d2h_bytes_per_step": B * sum(4 * m["rows"] for m in mats),
                "note": None if L == 1 else "one copy of the activations in, every layer's launches, one copy of the last layer's results out"},
        "decode_only": None if not decode_ms else {
            "ms_per_step": decode_ms, "uncompressed_GBs": unc_bytes / (decode_ms * 1e-3) / 1e9,
            "hbm_GBs_read_plus_written": (sum(m["blob_bytes"] for m in mats) + unc_bytes) / (decode_ms * 1e-3) / 1e9,
            "note": "huffllm_decode of every matrix of the step, one launch each, into a device buffer"},
        "gpu_launches": len(groups) * args.steps * R,
        "clocks": clocks,
        "split_explorer": explorer,
        "dense_bf16_gemv": {"own_kernel_ms_per_step": plain_ms, "cublas_mv_ms_per_step": cublas_ms,
                            "own_kernel_GBs": None if not plain_ms else unc_bytes / (plain_ms * 1e-3) / 1e9,
                            "own_kernel_frac_of_hbm_peak": None if not plain_ms else unc_bytes / (plain_ms * 1e-3) / 1e9 / peak,
                            "launches_per_step": len(groups),
                            "speedup_vs_own_dense": None if not plain_ms else plain_ms / ms_step,
                            "compression_ratio_total": unc_bytes / (L * sum(m["blob_bytes"] for m in mats)),
                            "note": "own streaming kernel in the same launch groups as the compressed path; the north star asks for "
                                    "speedup_vs_own_dense >= compression_ratio_total"},
        "small_batch": small_batch,
        "fp16": fp16_one,
        "sweep_8b_32_layers": sweep_8b,
        "cpu_baseline_all_cores": cpu_all,
        "timing": {"regions": R, "steps_per_region": args.steps, "ms_per_step_min": ms_min, "ms_per_step_median": ms_step,
                   "ms_per_step_max": ms_max, "note": "every region is exactly --steps steps between two CUDA events; the line's "
                                                       "ms_per_step and value are the median region"},
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
