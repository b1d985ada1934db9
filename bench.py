#!/usr/bin/env python
"""Decode-throughput benchmark of the fused EntroPack decoder on B200.

One "step" is one pass of the whole hot path (rANS decode -> E8 point -> row rescale -> dtype
store) over one workload.  Default workload: the 48-layer stack of transformer-block bundles at 3.5 bpp decoded layer by
layer into one reused BF16 buffer (config 5 of the baseline, the largest single-GPU configuration and one of the
two the roofline target is stated on); the other one, the 8192x8192 Laplace tensor at 4.0 bpp to FP16, is
--workload c4.  Other workloads: --workload c1 | c2 | c3.

  python bench.py [--gpus N --steps K --warmup W] [--workload c4 --bpp 4.0 --tile-vectors V]
  python bench.py --impl reference       # the CPU oracle on the same workload (bounded sample per step)

Prints ONE JSON line (rank 0).  Timing: CUDA events on the launching stream around each step, an
L2 flush (512 MB write) between steps outside the events, max over ranks.  After the headline measurement (and
outside its timed region) the default run also measures the other stated configurations and puts them in the
same line under "records": the 8192x8192 tensor at 4.0 bpp with its own roofline block, its rate sweep 2.0 .. 6.0,
the block bundle decoded to FP8-E4M3 and to INT8, the paper's default tile size, and one GPU-encoder call
(--no-extras skips them).

--gpus N > 1 without a launcher starts N ranks itself (torch.distributed.run on 127.0.0.1): independent replicas,
NCCL only for the barrier and the max-reduction of the times.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_HBM_GBS = 6650.0   # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent

# dram bytes (read + write) per launch measured with ncu for the default workload, filled in from
# profiles/ after a capture; None = not captured for this workload
NCU_TRAFFIC_BYTES = {("c4", 4.0, "fp16"): 39581696 + 76114944,      # dram read + write of one launch
                     ("c4", 8.0, "fp16"): 68460032 + 80646656,
                     ("c5", 3.5, "bf16"): 207602944 + 686487552}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--bpp", type=float, default=None, help="target bits/param (default: the workload's)")
    ap.add_argument("--tile-vectors", type=int, default=-1,
                    help="V; 0 = the paper's default for the target rate; -1 (default) = ep_suggest_tile_vectors[_batch]: "
                         "a V up to the paper's default that fills whole rounds of the GPU's tile slots")
    ap.add_argument("--dtype", default=None, choices=[None, "bf16", "fp16", "fp8", "int8"])
    ap.add_argument("--layers", type=int, default=48, help="c5: resident layers")
    ap.add_argument("--distinct-layers", type=int, default=2, help="c5: distinct layers actually encoded")
    ap.add_argument("--sweep", action="store_true",
                    help="c4 only: after the main line's measurement also time every target rate 2.0, 2.5 .. 6.0 "
                         "(throughput and stored vs target bpp per rate, in the JSON key 'sweep')")
    ap.add_argument("--gemm-curve", action="store_true",
                    help="also time decode-then-GEMM against a GEMM on resident BF16 weights (10240x3840 layer, 4 bpp)")
    ap.add_argument("--graph", action="store_true",
                    help="record the step's launches once in a CUDA graph and replay it in the timed region")
    ap.add_argument("--no-extras", action="store_true",
                    help="headline workload only: skip the records of the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


# ---- workloads ---------------------------------------------------------------------------------------

def make_workload(args, rows=None):
    """Returns (name, dtype_name, target_bpp, list of layers, full shapes of one layer); a layer is a list of fp32
    matrices.  rows: draw only that many rows of every tensor (same distribution and width; the CPU arm's sample)."""
    from paper_2609_34185_b200 import synth
    w = args.workload
    cut = (lambda R: R) if rows is None else (lambda R: min(R, rows))
    if w == "c4":
        return ("config4: 8192x8192 Laplace rows", args.dtype or "fp16", args.bpp or 4.0, [[synth.config4(R=cut(8192))]],
                [(8192, 8192)])
    if w == "c1":
        if args.tile_vectors < 0:
            args.tile_vectors = 4096            # the configuration fixes one tile per 64 rows
        return ("config1: 512x512 Gaussian rows, one tile per 64 rows", args.dtype or "bf16", args.bpp or 4.0,
                [[synth.config1()]], [(512, 512)])
    if w == "c2":
        return ("config2: 4096x4096 Student-t rows", args.dtype or "bf16", args.bpp or 3.0, [[synth.config2(R=cut(4096))]],
                [(4096, 4096)])
    if w == "c3":
        kind = args.dtype or "fp8"
        mats = [container_values(synth.config3_tensor(i, shape=(cut(R), C)), kind)[1] if kind in ("fp8", "int8")
                else synth.config3_tensor(i, shape=(cut(R), C)) for i, (R, C) in enumerate(synth.BLOCK_SHAPES)]
        return ("config3: block bundle 4x5120^2 + 3x5120x17408, 0.1% outliers", kind, args.bpp or 2.5, [mats],
                list(synth.BLOCK_SHAPES))
    if w == "c5":
        layers = [[synth.config5_tensor(l, i, shape=(cut(R), C)) for i, (R, C) in enumerate(synth.BLOCK_SHAPES)]
                  for l in range(args.distinct_layers if rows is None else 1)]
        return (f"config5: {args.layers}-layer stack of block bundles ({args.distinct_layers} distinct layers "
                f"encoded, cycled)"), args.dtype or "bf16", args.bpp or 3.5, layers, list(synth.BLOCK_SHAPES)
    raise ValueError(w)


def container_values(W, kind):
    """The FP8 / INT8 route (Sec. "FP8 and INT8 computation"): weights scaled row by row into the container and
    rounded to its grid; these values are what gets compressed.  Returns (per-row output scale, container values)."""
    from paper_2609_34185_b200 import synth
    a, Wc = synth.to_container(W, kind)
    if kind == "fp8":
        import torch
        return a, torch.from_numpy(Wc).to(torch.float8_e4m3fn).float().numpy()
    return a, np.clip(np.rint(Wc), -128, 127).astype(np.float32)


# tile-size suggestions in plain Python, for the CPU arm (which must not load the CUDA library): the same rules as
# ep_suggest_tile_vectors / ep_suggest_tile_vectors_batch with 32 tiles per SM (tests compare the two)
TILES_PER_SM = 32


def suggest_v_py(R, C, vmax, slots):
    nvec = R * (C // 8)
    if slots == 0 or nvec == 0:
        return vmax
    floor_v = max(32, vmax // 4 // 32 * 32)
    rounds = 1
    while True:
        tiles = rounds * slots
        V = -(-nvec // tiles)
        if V <= vmax:
            V32 = (V + 31) // 32 * 32
            if V32 <= vmax:
                V = V32
            return max(V, floor_v)
        rounds += 1


def suggest_v_batch_py(shapes, vmax, ctas):
    if not shapes or ctas == 0:
        return vmax
    lo = max(32, vmax // 4 // 32 * 32)
    best_v, best_cost = vmax, None
    for V in range(lo, vmax + 1, 32):
        rounds = sum(-(-(-(-(R * (C // 8)) // V)) // TILES_PER_SM) for R, C in shapes)
        cost = -(-rounds // ctas) * (V // 32 + 2)
        if best_cost is None or cost <= best_cost:
            best_cost, best_v = cost, V
    return best_v


def pick_tile_vectors(V, shape, bpp, slots, batch_shapes=None):
    """V < 0: a single tensor gets ep_suggest_tile_vectors for the GPU's tile slots; the tensors of a batch (decoded by
    one launch, `batch_shapes`) get ep_suggest_tile_vectors_batch for the GPU's SMs: one multiple of 32 up to the
    paper's default for which the rounds of all tensors split evenly over the CTAs."""
    import paper_2609_34185_b200 as ep
    if V >= 0:
        return V
    if batch_shapes is not None and len(batch_shapes) > 1:
        return ep.suggest_tile_vectors_batch(batch_shapes, bpp, slots // ep.decode_tiles_per_sm())
    return ep.suggest_tile_vectors(shape[0], shape[1], bpp, slots)


def encode_layers(layers, bpp, V, slots, dev=None):
    """Streams of the workload (set-up, untimed).  With a device the library's CUDA encoder back end is used - it
    gives the host encoder's bytes - and the host encoder serves whatever it declines."""
    import paper_2609_34185_b200 as ep
    out = []
    for mats in layers:
        shapes = [W.shape for W in mats]
        blobs = []
        for W in mats:
            tv = pick_tile_vectors(V, W.shape, bpp, slots, shapes)
            blob = None
            if dev is not None:
                import torch
                try:
                    blob = ep.encode_device(torch.from_numpy(W).to(dev), bpp, tile_vectors=tv)
                except ep.EntroPackError as e:
                    if e.status != -3:
                        raise
            blobs.append(blob if blob is not None else ep.encode(W, bpp, tile_vectors=tv))
        out.append(blobs)
    return out


# ---- clocks ------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "20"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def wait_first(self, timeout=5.0):
        t0 = time.time()
        while self.proc is not None and not self.lines and time.time() - t0 < timeout:
            time.sleep(0.01)

    def mark(self):
        """Index of the next sample: samples from here on were taken during the timed region."""
        return len(self.lines)

    def stop(self, start=0, min_samples=3):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        lines = self.lines[start:] if len(self.lines) - start >= min_samples else self.lines
        for ln in lines:
            p = [t.strip() for t in ln.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- CPU oracle legs -----------------------------------------------------------------------------------

ORACLE_DT = {"bf16": 0, "fp16": 1, "fp8": 2, "int8": 3}


def oracle_sample(blob, dtype_name, target_seconds=1.5):
    """Sizes a bounded sample of the oracle decoder's work on one stream: a leading tile range, repeated
    `reps` times, that takes about target_seconds.  Returns (params per repetition, tiles, reps, threads)."""
    import oracle
    I = blob.info
    n_tiles = I.n_tiles
    probe = max(1, min(n_tiles, 64))
    oracle.decode(blob.data, ORACLE_DT[dtype_name], tiles=(0, probe))       # also builds / loads the oracle
    t0 = time.perf_counter()
    oracle.decode(blob.data, ORACLE_DT[dtype_name], tiles=(0, probe))
    dt = max(time.perf_counter() - t0, 1e-4)
    want = probe * target_seconds / dt
    tiles = int(max(probe, min(n_tiles, want)))
    reps = int(max(1, min(200, want / tiles)))
    nvec = min(tiles * I.V, I.R * I.C // 8)
    return 8 * nvec, tiles, reps, oracle.num_threads()


def oracle_time(blob, dtype_name, tiles, reps):
    import oracle
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.decode(blob.data, ORACLE_DT[dtype_name], tiles=(0, tiles))
    return time.perf_counter() - t0


def run_reference(args):
    """The reference arm: the CPU oracle alone (encoder and decoder; the CUDA library is never loaded).  A step
    decodes a bounded sample of the workload: the first rows of every tensor of its first layer, compressed by
    the oracle's encoder at the workload's target rate and the GPU arm's tile size.  Rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    if os.environ.get("WORLD_SIZE") is not None:
        # a launcher pins OMP_NUM_THREADS to 1 for its ranks; this arm runs on rank 0 alone, so give it the host's cores
        oracle.set_threads(os.cpu_count() or 1)
    probe_rows = 64
    name, dtype_name, bpp, layers, shapes = make_workload(args, rows=probe_rows)
    vmax = oracle.default_tile_vectors(bpp)
    if args.tile_vectors >= 0:
        V = args.tile_vectors
    elif len(shapes) > 1:
        V = suggest_v_batch_py(shapes, vmax, 148)
    else:
        V = suggest_v_py(shapes[0][0], shapes[0][1], vmax, 148 * TILES_PER_SM)
    odt = ORACLE_DT[dtype_name]

    def encode_all(mats):
        return [oracle.encode(W, bpp, oracle.default_opts(tile_vectors=V))[0] for W in mats]

    def decode_all(blobs):
        t0 = time.perf_counter()
        for b in blobs:
            oracle.decode(b, odt)
        return time.perf_counter() - t0

    # size the sample: rows per tensor such that one step takes about the budget (whole run: about a minute)
    blobs = encode_all(layers[0])
    decode_all(blobs)
    dt = max(decode_all(blobs), 1e-4)
    budget = min(0.5, 60.0 / max(1, args.steps + args.warmup))
    rows = int(max(8, min(max(R for R, _ in shapes), probe_rows * budget / dt)))
    if rows != probe_rows:
        name, dtype_name, bpp, layers, shapes = make_workload(args, rows=rows)
        blobs = encode_all(layers[0])
    params = sum(W.size for W in layers[0])
    stored = 8.0 * sum(len(b) for b in blobs) / params
    times = []
    for i in range(args.warmup + args.steps):
        dt = decode_all(blobs)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = params * len(times) / total / 1e9
    threads = oracle.num_threads()
    sample = (f"oracle decoder on oracle-encoded streams of the first {rows} rows of each of the {len(blobs)} tensors of "
              f"the workload's first layer ({params} params per step)")
    line = {"impl": "reference", "metric": "decoded Gparams/s", "value": value, "unit": "Gparams/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype_name, "data": "synthetic",
            "config": {"workload": name, "target_bpp": bpp, "stored_bpp": stored, "tile_vectors": V,
                       "out_dtype": dtype_name, "params_per_step": params},
            "cpu_baseline": {"value": value, "unit": "Gparams/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "Gparams/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- the GPU arm ---------------------------------------------------------------------------------------

def decode_then_gemm_curve(ep, torch, dev, stream, flush, n_sms):
    """Overhead of reconstructing a layer before each use (the experiment of Sec. "Reconstruction cost and tile
    overhead", right panel): y = x W^T with W a 10240 x 3840 BF16 layer, x holding 256 .. 16384 tokens, once on
    resident dense weights and once as decode + the same product.  The product is the library's (torch.matmul);
    only the decode is this repository's kernel.  Median of 15 flushed repetitions each."""
    from paper_2609_34185_b200 import synth
    R, C, bpp = 10240, 3840, 4.0
    W = synth.gaussian_rows(R, C, 77)
    V = pick_tile_vectors(-1, W.shape, bpp, ep.decode_tiles_per_sm() * n_sms)
    blob = ep.encode(W, bpp, tile_vectors=V)
    d = ep.upload(blob, device=dev)
    Wd = torch.empty(R, C, dtype=torch.bfloat16, device=dev)
    ep.decode(d, ep.BF16, out=Wd, stream=stream)
    g = torch.Generator(device=dev)
    g.manual_seed(78)

    def median_ms(fn):
        for _ in range(3):
            fn()
        ts = []
        for _ in range(15):
            flush.fill_(0)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    rows = []
    for tokens in (256, 1024, 4096, 16384):
        x = torch.randn(tokens, C, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        y = torch.empty(tokens, R, dtype=torch.bfloat16, device=dev)

        def dense():
            torch.matmul(x, Wd.t(), out=y)

        def with_decode():
            ep.decode(d, ep.BF16, out=Wd, stream=stream)
            torch.matmul(x, Wd.t(), out=y)

        t_dense, t_both = median_ms(dense), median_ms(with_decode)
        rows.append({"tokens": tokens, "gemm_ms": t_dense, "decode_gemm_ms": t_both,
                     "overhead_pct": 100.0 * (t_both - t_dense) / t_dense})
        del x, y
    return {"layer": [R, C], "target_bpp": bpp, "stored_bpp": blob.stored_bpp, "tile_vectors": blob.info.V,
            "rows": rows}



def timed_flushed(torch, stream, flush, fn, reps=24, warm=3):
    """(min, mid-mean) in ms of `reps` runs of fn, each after an L2 flush, CUDA events on `stream`."""
    for _ in range(warm):
        fn()
    ts = []
    for _ in range(reps):
        flush.fill_(0)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    # event times of one short launch come in steps of about 2 us on this GPU: the mean of the central half of
    # the sorted times resolves what the median cannot
    ts.sort()
    mid = ts[len(ts) // 4: len(ts) - len(ts) // 4]
    return min(ts), sum(mid) / len(mid)


def fused_gemm_record(ep, torch, dev, stream, timed, slots):
    """The decode fused into the matrix product (ep_decode_gemm) on the 10240 x 3840 layer of the reconstruction-cost
    experiment: up to 32 tokens, against decoding (with the decode path's own tile size) and multiplying with
    torch.matmul.  `timed(fn)` returns (min, mid-mean) of flushed repetitions in ms."""
    from paper_2609_34185_b200 import synth
    Wl = torch.from_numpy(synth.gaussian_rows(10240, 3840, 77)).to(dev)
    bl_row = ep.encode_device(Wl, 4.0, tile_vectors=3840 // 8)            # one tile per row: the layout the fused kernel reads
    bl_dec = ep.encode_device(Wl, 4.0, tile_vectors=ep.suggest_tile_vectors(10240, 3840, 4.0, slots))
    d_row, d_dec = ep.upload(bl_row, device=dev), ep.upload(bl_dec, device=dev)
    wbuf = torch.empty((10240, 3840), dtype=torch.bfloat16, device=dev)
    rows = []
    gen = torch.Generator(device=dev)
    gen.manual_seed(78)
    for tokens in (8, 16, 32):
        x = torch.randn(tokens, 3840, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        y32 = torch.empty((tokens, 10240), dtype=torch.float32, device=dev)
        y16 = torch.empty((tokens, 10240), dtype=torch.bfloat16, device=dev)

        def two_kernels():
            ep.decode(d_dec, ep.BF16, out=wbuf, stream=stream)
            torch.matmul(x, wbuf.t(), out=y16)

        _, t_two = timed(two_kernels)
        _, t_fused = timed(lambda: ep.decode_matmul(d_row, x, out=y32, stream=stream))
        rows.append({"tokens": tokens, "decode_then_matmul_ms": t_two, "fused_ms": t_fused})
        del x, y32, y16
    return {"rows": rows, "stored_bpp_fused_layout": bl_row.stored_bpp, "stored_bpp_decode_layout": bl_dec.stored_bpp,
            "tile_vectors_decode_layout": bl_dec.info.V,
            "what": "y = x W^T, W a 10240 x 3840 layer at 4 bpp: ep_decode_gemm (weights never written to memory) "
                    "against ep_decode_batch + torch.matmul"}


def peak_info():
    """(HBM GB/s the roofline fractions refer to, where the number comes from)"""
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def extra_records(ep, torch, dev, stream, flush, slots, n_sms, peak, skip):
    """The stated configurations other than the headline one, each timed as the paper times its codec (CUDA events
    around the call, three warm-ups, then repeated runs; here 24 runs with an L2 flush before each, the mean of the
    central half reported).  Streams come from the library's GPU encoder (byte-identical to the host encoder's).
    Returns a dict of records."""
    from paper_2609_34185_b200 import synth

    def timed(fn, reps=24, warm=3):
        return timed_flushed(torch, stream, flush, fn, reps, warm)

    def record(params, nbytes_in, esize, ms, **more):
        alg = nbytes_in + params * esize
        gbs = alg / (ms * 1e-3) / 1e9
        return dict(Gparams_per_s=params / (ms * 1e-3) / 1e9, midmean_ms=ms, effective_GBps=gbs,
                    roofline={"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                              "bytes_per_launch": alg, "ms_per_launch": ms, "kernel": "ep_decode_smem_kernel"}, **more)

    out = {}
    # ---- config 4: 8192 x 8192 Laplace rows to FP16, 4.0 bpp and the sweep 2.0 .. 6.0 ----
    W4 = torch.from_numpy(synth.config4()).to(dev)
    buf = torch.empty((8192, 8192), dtype=torch.float16, device=dev)
    sweep = []
    for r in (2.0, 2.5, 3.0, 3.5, 4.0, 4.5, 5.0, 5.5, 6.0):
        V = ep.suggest_tile_vectors(8192, 8192, r, slots)
        bl = ep.encode_device(W4, r, tile_vectors=V)
        dd = ep.upload(bl, device=dev)
        mn, med = timed(lambda: ep.decode(dd, ep.FP16, out=buf, stream=stream))
        rec = record(W4.numel(), len(bl), 2, med, target_bpp=r, stored_bpp=bl.stored_bpp, tile_vectors=bl.info.V,
                     b=bl.info.b, min_ms=mn)
        sweep.append(rec)
        if r == 4.0:
            out["config4_fp16_4.0bpp"] = dict(rec, traffic=NCU_TRAFFIC_BYTES.get(("c4", 4.0, "fp16")))
            # the paper's default tile size for this rate (not a multiple of 32: the last group of every tile is
            # partly filled) against the suggested one
            blp = ep.encode_device(W4, r, tile_vectors=ep.default_tile_vectors(r))
            dp = ep.upload(blp, device=dev)
            mnp, medp = timed(lambda: ep.decode(dp, ep.FP16, out=buf, stream=stream))
            out["config4_fp16_4.0bpp_paper_tile_size"] = record(W4.numel(), len(blp), 2, medp, target_bpp=r,
                                                                stored_bpp=blp.stored_bpp, tile_vectors=blp.info.V, min_ms=mnp)
            del dp
        del dd
    # the paper's other headline rate: 8 bpp (b = 12, two-level lookup tables)
    V8 = ep.suggest_tile_vectors(8192, 8192, 8.0, slots)
    bl8 = ep.encode_device(W4, 8.0, tile_vectors=V8)
    d8 = ep.upload(bl8, device=dev)
    mn8, med8 = timed(lambda: ep.decode(d8, ep.FP16, out=buf, stream=stream))
    out["config4_fp16_8.0bpp"] = dict(record(W4.numel(), len(bl8), 2, med8, target_bpp=8.0, stored_bpp=bl8.stored_bpp,
                                             tile_vectors=bl8.info.V, b=bl8.info.b, min_ms=mn8),
                                      traffic=NCU_TRAFFIC_BYTES.get(("c4", 8.0, "fp16")))
    del d8
    out["config4_sweep_fp16"] = [{k: v for k, v in rec.items() if k != "roofline"} | {"frac": rec["roofline"]["frac"]}
                                 for rec in sweep]
    # one call of the GPU encoder on the same tensor (wall time of the call, buffers warm)
    ws = None
    for _ in range(2):
        t0 = time.perf_counter()
        bl = ep.encode_device(W4, 4.0, tile_vectors=ep.suggest_tile_vectors(8192, 8192, 4.0, slots))
        enc_ms = 1e3 * (time.perf_counter() - t0)
    out["encode_device_8192x8192_4.0bpp"] = {"ms": enc_ms, "stored_bpp": bl.stored_bpp,
                                             "what": "ep_encode_device call to finished host blob, second call"}
    del W4, buf
    out["decode_gemm_10240x3840_4.0bpp"] = fused_gemm_record(ep, torch, dev, stream, timed, slots)
    # ---- config 3: the block bundle in its FP8-E4M3 and INT8 containers, 2.5 bpp, one batched launch ----
    if skip != "c3":
        V = ep.suggest_tile_vectors_batch(synth.BLOCK_SHAPES, 2.5, n_sms)
        src = [synth.config3_tensor(i) for i in range(7)]
        for kind, DT, tdt in (("fp8", ep.FP8_E4M3, torch.float8_e4m3fn), ("int8", ep.INT8, torch.int8)):
            blobs = [ep.encode_device(torch.from_numpy(container_values(W, kind)[1]).to(dev), 2.5, tile_vectors=V) for W in src]
            total = sum(b.info.R * b.info.C for b in blobs)
            obuf = torch.empty(total, dtype=tdt, device=dev)
            outs, at = [], 0
            for b in blobs:
                n = b.info.R * b.info.C
                outs.append(obuf[at:at + n].view(b.info.R, b.info.C))
                at += n
            ds = [ep.upload(b, device=dev) for b in blobs]
            mn, med = timed(lambda: ep.decode_many(ds, DT, outs, stream=stream))
            nin = sum(len(b) for b in blobs)
            out[f"config3_{kind}_2.5bpp"] = record(total, nin, 1, med, target_bpp=2.5, stored_bpp=8.0 * nin / total,
                                                   tile_vectors=V, min_ms=mn, launches=1)
            del ds, obuf, outs, blobs
    if ep.last_device_status() != 0:
        raise RuntimeError("decoder reported an inconsistent stream in the extra records")
    return out


def main():
    args = parse_args()
    env_world = os.environ.get("WORLD_SIZE")
    if args.gpus > 1 and env_world is None:
        # no launcher: start the N ranks ourselves, one process per GPU, rendezvous on the loopback address
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if env_world is not None and int(env_world) != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {env_world} ranks", file=sys.stderr)
        sys.exit(2)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2609_34185_b200 as ep

    ep.load()   # fails loudly if the CUDA library is missing: there is no fallback
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    name, dtype_name, bpp, layers, _shapes = make_workload(args)
    DT = {"bf16": ep.BF16, "fp16": ep.FP16, "fp8": ep.FP8_E4M3, "int8": ep.INT8}[dtype_name]
    tdt = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp8": torch.float8_e4m3fn, "int8": torch.int8}[dtype_name]
    esize = ep.DTYPE_BYTES[DT]

    # every rank decodes its own replica of the workload: tiles and tensors are independent, no collective
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    # one persistent CTA per SM, ep_decode_tiles_per_sm() tiles in flight each
    slots = ep.decode_tiles_per_sm() * n_sms
    blobs = encode_layers(layers, bpp, args.tile_vectors, slots, dev)
    n_layers = args.layers if args.workload == "c5" else len(blobs)
    resident = [[ep.upload(b, device=dev) for b in blobs[l % len(blobs)]] for l in range(n_layers)]
    layer_params = [sum(b.info.R * b.info.C for b in blobs[l % len(blobs)]) for l in range(n_layers)]
    layer_bytes_in = [sum(len(b) for b in blobs[l % len(blobs)]) for l in range(n_layers)]
    params_per_step = sum(layer_params)
    comp_bytes_per_step = sum(layer_bytes_in)
    out_bytes_layer = max(layer_params) * esize
    out_buf = torch.empty(max(layer_params), dtype=tdt, device=dev)     # one reused layer buffer

    def layer_outs(l):
        outs, at = [], 0
        for d in resident[l]:
            n = d.info.R * d.info.C
            outs.append(out_buf[at:at + n].view(d.info.R, d.info.C))
            at += n
        return outs

    outs_by_layer = [layer_outs(l) for l in range(n_layers)]
    launches_per_step = sum((len(r) + ep.binding.MAX_BATCH - 1) // ep.binding.MAX_BATCH for r in resident)
    stream = torch.cuda.current_stream()

    def decode_layer(l, st=None):
        st = stream if st is None else st
        if len(resident[l]) == 1:
            ep.decode(resident[l][0], DT, out=outs_by_layer[l][0], stream=st)
        else:
            ep.decode_many(resident[l], DT, outs_by_layer[l], stream=st)

    def step(st=None):
        for l in range(n_layers):
            decode_layer(l, st)

    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_first()
    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    barrier()
    if ep.last_device_status() != 0:
        raise RuntimeError("decoder reported an inconsistent stream during warm-up")
    barrier()
    run_step = step
    if args.graph:
        graph = torch.cuda.CUDAGraph()
        cap = torch.cuda.Stream(device=dev)
        cap.wait_stream(stream)
        with torch.cuda.stream(cap):
            with torch.cuda.graph(graph, stream=cap):
                step(cap)
        stream.wait_stream(cap)
        run_step = graph.replay
        for _ in range(2):
            run_step()
        barrier()
    mark = sampler.mark()
    evs = []
    for _ in range(args.steps):
        flush.fill_(0)      # L2 flush between timed iterations, outside the events
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(stream)
        run_step()
        e.record(stream)
        evs.append((s, e))
    barrier()
    clocks = sampler.stop(mark) if rank == 0 else None
    times_ms = [s.elapsed_time(e) for s, e in evs]
    # the same steps back to back without the flush ("warm": a stream smaller than L2 stays cached); reported beside
    # the flushed figure, never used for the roofline claim
    ws, we = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    warm_steps = max(3, min(args.steps, 50))
    ws.record(stream)
    for _ in range(warm_steps):
        step()
    we.record(stream)
    barrier()
    warm_ms = ws.elapsed_time(we) / warm_steps
    total_ms = sum(times_ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * params_per_step / (ms_per_step * 1e-3) / 1e9           # Gparams/s, whole job
    alg_bytes_step = comp_bytes_per_step + params_per_step * esize
    eff_gbs = alg_bytes_step / (ms_per_step * 1e-3) / 1e9                  # per GPU

    # end to end through the public call with host buffers: pinned blob -> device, decode, result -> pinned host
    e2e = None
    if not args.no_e2e:
        l0 = 0
        # two slots, each with its own stream and buffers: the copy-in of one step overlaps the copy-out of the one
        # before (PCIe is full duplex); every step still moves its whole input and its whole result
        n_slots = 2
        pinned_in = [torch.from_numpy(b.data).pin_memory() for b in blobs[l0]]
        slot_stream = [torch.cuda.Stream(device=dev) for _ in range(n_slots)]
        slot_in = [[torch.empty(len(b), dtype=torch.uint8, device=dev) for b in blobs[l0]] for _ in range(n_slots)]
        slot_dev_out = [torch.empty(layer_params[l0], dtype=tdt, device=dev) for _ in range(n_slots)]
        slot_host_out = [torch.empty(layer_params[l0], dtype=tdt).pin_memory() for _ in range(n_slots)]
        # (the stream arrives anew in every step: its lookup tables are derived inside the decode, not prepared ahead)
        slot_scratch = [[ep.DeviceBlob(d, b.info, prepare=False) for d, b in zip(slot_in[k], blobs[l0])] for k in range(n_slots)]
        slot_outs = []
        for k in range(n_slots):
            outs, at = [], 0
            for b in blobs[l0]:
                n = b.info.R * b.info.C
                outs.append(slot_dev_out[k][at:at + n].view(b.info.R, b.info.C))
                at += n
            slot_outs.append(outs)
        h2d = sum(len(b) for b in blobs[l0])
        d2h = layer_params[l0] * esize
        e2e_steps = max(4, min(args.steps, 20))

        def e2e_step(i):
            k = i % n_slots
            st = slot_stream[k]
            with torch.cuda.stream(st):
                for p, d in zip(pinned_in, slot_in[k]):
                    d.copy_(p, non_blocking=True)
                ds = slot_scratch[k]
                if len(ds) == 1:
                    ep.decode(ds[0], DT, out=slot_outs[k][0], stream=st)
                else:
                    ep.decode_many(ds, DT, slot_outs[k], stream=st)
                slot_host_out[k].copy_(slot_dev_out[k], non_blocking=True)

        for i in range(4):
            e2e_step(i)
        barrier()
        t0 = time.perf_counter()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(stream)
        for st in slot_stream:
            st.wait_stream(stream)
        for i in range(e2e_steps):
            e2e_step(i)
        for st in slot_stream:
            stream.wait_stream(st)
        e.record(stream)
        barrier()
        ms = s.elapsed_time(e) / e2e_steps
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        e2e = {"value": world * layer_params[l0] / (ms * 1e-3) / 1e9, "unit": "Gparams/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms,
               "what": ("one layer per step: pinned host blob -> device, decode, decoded tensor -> pinned host; "
                        "two steps in flight on two streams")}
        del slot_in, slot_dev_out, slot_host_out, slot_scratch

    # per-layer device times of one more pass (config 5 asks for total and per-layer decode time)
    per_layer_ms = None
    if n_layers > 1:
        pev = [torch.cuda.Event(enable_timing=True) for _ in range(n_layers + 1)]
        pev[0].record(stream)
        for l in range(n_layers):
            decode_layer(l)
            pev[l + 1].record(stream)
        barrier()
        per_layer_ms = [pev[l].elapsed_time(pev[l + 1]) for l in range(n_layers)]

    # relative L2 error of the decoded first tensor against its source (Eq. 1; reporting only, torch fp64 on the GPU)
    d0, W0 = resident[0][0], torch.from_numpy(layers[0][0]).to(dev)
    got0 = ep.decode(d0, DT, out=outs_by_layer[0][0], stream=stream)
    torch.cuda.synchronize()
    g64, w64 = got0.to(torch.float64), W0.to(torch.float64)
    rel_l2_first = float(torch.sqrt(((g64 - w64) ** 2).sum() / (w64 ** 2).sum()).item())
    del g64, w64, W0

    sweep = None
    if args.sweep and args.workload == "c4" and rank == 0:
        sweep = []
        W = layers[0][0]
        for r in (2.0, 2.5, 3.0, 3.5, 4.0, 4.5, 5.0, 5.5, 6.0):
            V = pick_tile_vectors(args.tile_vectors, W.shape, r, slots)
            bl = ep.encode(W, r, tile_vectors=V)
            dd = ep.upload(bl, device=dev)
            for _ in range(3):
                ep.decode(dd, DT, out=outs_by_layer[0][0], stream=stream)
            ts = []
            for _ in range(15):                      # the paper's protocol: minimum of fifteen after three warm-ups
                flush.fill_(0)
                a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                ep.decode(dd, DT, out=outs_by_layer[0][0], stream=stream)
                b_.record(stream)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b_))
            med = statistics.median(ts)
            nbytes = len(bl) + W.size * esize
            sweep.append({"target_bpp": r, "stored_bpp": bl.stored_bpp, "tile_vectors": bl.info.V, "min_ms": min(ts),
                          "median_ms": med, "Gparams_per_s": W.size / (med * 1e-3) / 1e9,
                          "effective_GBps": nbytes / (med * 1e-3) / 1e9})
            del dd

    gemm_curve = None
    if args.gemm_curve and rank == 0:
        gemm_curve = decode_then_gemm_curve(ep, torch, dev, stream, flush, n_sms)
        gemm_curve["fused"] = fused_gemm_record(ep, torch, dev, stream,
                                                lambda fn: timed_flushed(torch, stream, flush, fn), slots)


    records = None
    if not args.no_extras and rank == 0:
        records = extra_records(ep, torch, dev, stream, flush, slots, n_sms, peak_info()[0], skip=args.workload)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = peak_info()
    # dominant (only) kernel: the fused decode; algorithmic bytes per launch = compressed bytes + weight bytes
    launch_bytes = alg_bytes_step / launches_per_step
    launch_ms = ms_per_step / launches_per_step
    achieved = launch_bytes / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES.get((args.workload, bpp, dtype_name)), "peak_source": peak_src,
                "kernel": "ep_decode_smem_kernel", "bytes_per_launch": launch_bytes, "ms_per_launch": launch_ms}

    cpu = None
    if not args.no_cpu_baseline:
        b0 = blobs[0][0]
        p, tiles, reps, threads = oracle_sample(b0, dtype_name, 2.0)
        dt = oracle_time(b0, dtype_name, tiles, reps)
        import oracle
        oracle.set_threads(1)
        one_tiles = max(1, tiles // max(1, threads))
        dt1 = oracle_time(b0, dtype_name, one_tiles, 1)
        oracle.set_threads(threads)
        p1 = 8 * min(one_tiles * b0.info.V, b0.info.R * b0.info.C // 8)
        cpu = {"value": p * reps / dt / 1e9, "unit": "Gparams/s", "cores": threads, "kind": "oracle",
               "sample": (f"oracle decoder on tiles 0..{tiles} of {b0.info.n_tiles} of the first tensor, {reps} times "
                          f"({p * reps} params, {dt:.2f} s wall)"),
               "one_core_value": p1 / dt1 / 1e9}

    b0 = blobs[0][0]
    stored = 8.0 * comp_bytes_per_step / params_per_step
    line = {"metric": "decoded Gparams/s", "value": value, "unit": "Gparams/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype_name, "data": "synthetic",
            "config": {"workload": name, "target_bpp": bpp, "stored_bpp": stored, "tile_vectors": b0.info.V,
                       "tiles_first_tensor": b0.info.n_tiles, "b": b0.info.b, "out_dtype": dtype_name,
                       "params_per_step": params_per_step, "l2": "flushed between timed steps (512 MB write)",
                       "launch": "cuda graph replay" if args.graph else "direct",
                       "min_ms": min(times_ms), "median_ms": statistics.median(times_ms),
                       "warm_ms_per_step_no_flush": warm_ms, "rel_l2_first_tensor": rel_l2_first},
            "effective_GBps": eff_gbs, "pct_of_measured_hbm": 100.0 * eff_gbs / peak, "pct_of_8TBps": 100.0 * eff_gbs / 8000.0,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "per_layer_ms": per_layer_ms, "sweep": sweep, "decode_then_gemm": gemm_curve, "records": records,
            "clocks": clocks}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
