#!/usr/bin/env python
"""Benchmark of the NVFP4 linear path on FLUX.1-shaped layers (one B200 per rank).

One "step" = the whole hot path over one batch: for each of the six FLUX.1 linears
(M = 8 samples x 4608 tokens) the dynamic per-tensor scale, the activation quantizer and the
block-scaled FP4 GEMM with BF16 output (weights are quantized once, outside the timed region,
as they change once per policy update).  The same layers then run through the BF16 tcgen05
GEMM to give the FP4-over-BF16 speedup on our own kernels.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "nvfp4_linear_tflops_flux_shapes"
UNIT = "TFLOP/s"
NOMINAL_FP4_TFLOPS = 9000.0     # vendor dense NVFP4 peak
NOMINAL_BF16_TFLOPS = 2250.0    # vendor dense BF16 peak
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (None until a capture of the current kernel exists)
# ncu capture of one d_proj launch (summaries under profiles/): GEMM 69.1 MB read + 171.6 MB
# written for 295.5 MB algorithmic (Y partly still dirty in L2 at kernel end); quantizer 226.5 + 26.5 MB
# for 290.2 MB algorithmic.  Scaled to all six layers by the algorithmic bytes (traffic is proportional).
NCU_TRAFFIC_RATIO = {"gemm": (69.06 + 171.63) / 295.5, "quantize": (226.53 + 26.43) / 290.2}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Logs SM clocks and throttle reasons with nvidia-smi (read-only) for the whole run, time-stamped, so
    that every timed region can be given the samples that fall inside it."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.log = None
        self.samples = []

    def start(self):
        import tempfile
        try:
            self.log = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.log, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        import datetime
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            self.proc.wait()
        self.log.flush()
        self.log.seek(0)
        for line in self.log.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                t = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                sm, mx, pw = float(f[1]), float(f[2]), float(f[3])
            except ValueError:
                continue
            self.samples.append((t, sm, mx, pw, {n for n, v in zip(self.NAMES, f[4:8]) if v.lower().startswith("active")}))
        self.log.close()
        try:
            os.unlink(self.log.name)
        except OSError:
            pass
        self.proc = None

    def window(self, windows):
        """Statistics of the samples inside the given (start, end) wall-clock windows (a margin of 60 ms is
        cut from both ends: nvidia-smi stamps a sample when it starts the query)."""
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sel = [x for x in self.samples if any(w0 + 0.06 <= x[0] <= w1 - 0.06 for w0, w1 in windows)]
        sm = [x[1] for x in sel]
        reasons = set()
        for x in sel:
            reasons |= x[4]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_mhz_min": min(sm) if sm else None,
                "sm_max_mhz": max(x[2] for x in self.samples), "power_w_max": max((x[3] for x in sel), default=None),
                "samples": len(sm), "reasons": sorted(reasons)}


def rolled_scale(B, torch, amax):
    """T for a running amax word, derived by the library's own kernel (sol_roll_tensor_scale)."""
    state = torch.zeros(2, dtype=torch.float32, device=amax.device)
    state[1:].copy_(amax)
    B.sol_roll_tensor_scale(state)
    return state[:1].clone()


def flops_of(layers) -> float:
    return float(sum(2.0 * l.M * l.N * l.K for l in layers))


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_tflops(cfg, layer_index: int, rows: int):
    """Times the oracle (quantize + FP64 dequantized matmul) on `rows` rows of one layer."""
    import numpy as np
    import oracle
    from paper_2604_06916_b200 import workloads

    layer = cfg.layers[layer_index]
    X, W, bias = workloads.make_layer(cfg, layer_index, "cpu", M=rows)
    xb, wb, bb = workloads.to_bits(X), workloads.to_bits(W), workloads.to_bits(bias)
    Tw = oracle.tensor_scale(wb)
    qw, sfw = oracle.quantize(wb, Tw)         # weights: outside the timed region, like the GPU arm
    t0 = time.perf_counter()
    Tx = oracle.tensor_scale(xb)
    qx, sfx = oracle.quantize(xb, Tx)
    Y = oracle.nvfp4_linear(qx, sfx, Tx, qw, sfw, Tw, bb)
    dt = time.perf_counter() - t0
    assert np.isfinite(Y).all()
    flops = 2.0 * rows * layer.N * layer.K
    return flops / dt / 1e12, dt, oracle.num_threads(), f"{rows} rows of {cfg.name}/{layer.name} (N={layer.N}, K={layer.K})"


def calibrated_rows(cfg, layer_index: int, target_s: float, fixed: int) -> int:
    """Rows of the sample so that one oracle pass takes about target_s on this host."""
    if fixed > 0:
        return fixed
    _, dt, _, _ = oracle_sample_tflops(cfg, layer_index, 256)
    rows = int(256 * target_s / max(dt, 1e-3))
    return max(256, min(cfg.layers[layer_index].M, (rows // 128) * 128))


def oracle_layer_on_rows(x_rows_bits, T_full, w_bits, bias_bits, M_full):
    """The oracle's stack (tensor scale, quantizer, FP64 matmul) timed on a row sample of one layer.

    The weights are quantized outside the timed part, as in the GPU arm.  `T_full` (the tensor scale of the
    whole activation tensor, or None) replaces the sample's own scale in the quantizer so that the result
    can be compared with the GPU's output rows; the scale pass over the sample is timed either way.
    Returns (Y, record) with the measured seconds, MAC count and the full-shape time extrapolated by rows.
    """
    import oracle

    Tw = oracle.tensor_scale(w_bits)
    qw, sfw = oracle.quantize(w_bits, Tw)
    rows, K = x_rows_bits.shape
    N = w_bits.shape[0]
    t0 = time.perf_counter()
    T_sample = oracle.tensor_scale(x_rows_bits)
    T = T_sample if T_full is None else T_full
    qx, sfx = oracle.quantize(x_rows_bits, T)
    Y = oracle.nvfp4_linear(qx, sfx, T, qw, sfw, Tw, bias_bits)
    dt = time.perf_counter() - t0
    macs = float(rows) * N * K
    rec = {"rows": int(rows), "seconds": round(dt, 3), "macs": macs, "gflops": round(2.0 * macs / dt / 1e9, 2),
           "full_shape_seconds_extrapolated": round(dt * M_full / rows, 1)}
    return Y, rec


def cpu_baseline_on_row_samples(B, torch, workloads, cfg, data, which: str):
    """CPU baseline: the oracle on the first configuration in full and, for each layer of the benchmark's
    workload, on the row sample the parity tests use (both end tiles + one row of every other tile, all N
    columns), with the full-shape time extrapolated by the row ratio.  The same rows of the GPU's output are
    compared with the oracle's (max error over tolerance per layer).  `which` = "all" adds the other
    model-shaped configurations and the sweep sizes (timing only, inputs generated on the device)."""
    import numpy as np
    import oracle

    t_all0 = time.perf_counter()
    out = {"unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "per_layer": []}
    # configuration 1 in full
    X1, W1, b1 = workloads.make_layer(workloads.CONFIG_SINGLE, 0, "cpu")
    _, rec = oracle_layer_on_rows(workloads.to_bits(X1), None, workloads.to_bits(W1), workloads.to_bits(b1), X1.shape[0])
    rec.update({"config": workloads.CONFIG_SINGLE.name, "layer": "lin", "full": True})
    rec.pop("full_shape_seconds_extrapolated")
    out["config1_full"] = rec
    tot_s = tot_macs = 0.0
    worst = 0.0
    for i, d in enumerate(data):
        l = d["l"]
        rows = workloads.sample_rows(l.M, seed=i)
        rows_t = torch.from_numpy(rows).to(d["X"].device)
        T_full = oracle.tensor_scale(workloads.to_bits(d["X"]))          # whole tensor (untimed: host copy of X)
        B.nvfp4_quantize_linear(d["X"], d["wq"], d["wsf"], d["wts"], d["bias"], workspace=d["ws"], out=d["Y"])
        y_gpu = oracle.bits_to_f64(workloads.to_bits(d["Y"][rows_t]))
        Y, rec = oracle_layer_on_rows(workloads.to_bits(d["X"][rows_t]), T_full, workloads.to_bits(d["W"]),
                                      workloads.to_bits(d["bias"]), l.M)
        ratio = float(np.max(np.abs(y_gpu - Y) / np.maximum(oracle.linear_tolerance(Y), 1e-300)))
        worst = max(worst, ratio)
        rec.update({"config": cfg.name, "layer": l.name, "oracle_max_err_over_tol": round(ratio, 4)})
        out["per_layer"].append(rec)
        tot_s += rec["seconds"]
        tot_macs += rec["macs"]
    out["value"] = 2.0 * tot_macs / tot_s / 1e12
    out["seconds"] = round(tot_s, 2)
    out["oracle_max_err_over_tol"] = round(worst, 4)
    out["step_seconds_extrapolated"] = round(sum(r["full_shape_seconds_extrapolated"] for r in out["per_layer"]), 1)
    out["sample"] = (f"{cfg.name}: {sum(r['rows'] for r in out['per_layer'])} rows over {len(data)} layers (both end tiles + one "
                     f"row of every other 128-row tile, all N columns), {tot_macs:.3g} MAC; configuration 1 in full")
    if which == "all":
        others = [workloads.CONFIG_SANA, workloads.CONFIG_SD35] + [workloads.config_sweep(g) for g in workloads.SWEEP_GROUPS]
        out["other_configs"] = []
        for c in others:
            if c.name == cfg.name:
                continue
            for i, l in enumerate(c.layers):
                X, W, bias = workloads.make_layer(c, i, data[0]["X"].device)
                rows_t = torch.from_numpy(workloads.sample_rows(l.M, seed=i)).to(X.device)
                _, rec = oracle_layer_on_rows(workloads.to_bits(X[rows_t]), None, workloads.to_bits(W),
                                              workloads.to_bits(bias), l.M)
                rec.update({"config": c.name, "layer": l.name})
                out["other_configs"].append(rec)
                del X, W, bias
    out["wall_seconds"] = round(time.perf_counter() - t_all0, 1)
    return out


def attention_numbers(B, n_s, seq, heads, loop_ms, peaks, peak_src):
    """Ours against torch's scaled-dot-product attention on one fused q/k/v projection output."""
    import torch
    import torch.nn.functional as F
    from paper_2604_06916_b200 import workloads
    _, q, k, v = workloads.make_qkv(n_s, seq, heads, 3, "cuda")
    out = torch.empty((n_s, seq, heads, 128), dtype=torch.bfloat16, device="cuda")
    t_ours = loop_ms(lambda: B.sol_attention_bf16(q, k, v, out=out))
    qt, kt, vt = q.transpose(1, 2), k.transpose(1, 2), v.transpose(1, 2)
    t_lib = loop_ms(lambda: F.scaled_dot_product_attention(qt, kt, vt))
    fl = 4.0 * n_s * heads * seq * seq * 128
    tf = fl / (t_ours * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    return {"shape": {"samples": n_s, "tokens": seq, "heads": heads, "head_dim": 128}, "ms": t_ours, "tflops": tf,
            "torch_sdpa_ms": t_lib, "torch_sdpa_tflops": fl / (t_lib * 1e-3) / 1e12,
            "roofline": {"bound": "tensor", "kernel": "attention_kernel", "achieved": tf, "peak": peak, "unit": "TFLOP/s",
                         "frac": tf / peak, "traffic": None,
                         "peak_source": peak_src + " (bf16 burst); the softmax's 2 x 16 K exponentials per tile on the SFU "
                                                   "(16 per clock per SM) take as long as the tile's MMAs"}}


def run_reference(args):
    from paper_2604_06916_b200 import workloads

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workloads.CONFIG_FLUX
    vals, secs = [], []
    sample = ""
    cores = 1
    rows = calibrated_rows(cfg, 1, 3.0, args.ref_rows)
    for i in range(args.warmup + args.steps):
        v, dt, cores, sample = oracle_sample_tflops(cfg, 1, rows)
        if i >= args.warmup:
            vals.append(v)
            secs.append(dt)
    value = sum(vals) / len(vals) if vals else 0.0
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / max(1, len(secs)), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "note": "CPU oracle on a bounded row sample of one layer per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU arm
class LegTimer:
    """Times named legs in long contiguous regions, rotated so that no leg always follows the same one.

    A leg's region repeats its K-step block until the region has run for at least `min_s` seconds (the
    GPU then sits in its power-capped steady state), with one CUDA event per block on the launching
    stream; regions are bracketed by barrier + synchronize and the per-step time is the max over ranks.
    Each of `rounds` rounds visits every leg once and starts at a different leg.
    """

    def __init__(self, torch, replicas, dev, dist, sampler, steps, min_s, rounds):
        self.torch, self.replicas, self.dev, self.dist = torch, replicas, dev, dist
        self.sampler, self.steps, self.min_s, self.rounds = sampler, steps, min_s, rounds
        self.nvtx = os.environ.get("SOL_BENCH_NVTX", "0") not in ("", "0")

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def region(self, fn, blocks):
        torch = self.torch
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
        self.barrier()
        w0 = time.time()
        ev[0].record()
        for b in range(blocks):
            for _ in range(self.steps):
                fn()
            ev[b + 1].record()
        self.barrier()
        w1 = time.time()
        total_ms = ev[0].elapsed_time(ev[-1])
        ms, _, _ = self.replicas.aggregate(total_ms / (blocks * self.steps), 1.0, self.dev)  # max over ranks
        return ms, total_ms * 1e-3, (w0, w1)

    def run(self, legs, warmup):
        """legs: ordered {name: fn}.  Returns {name: {ms_per_step (mean over rounds), per_round, spread, blocks,
        region_s, clocks}}."""
        names = list(legs)
        blocks = {}
        for n in names:                       # warm-up, and the block count that makes a region >= min_s
            for _ in range(warmup):
                legs[n]()
            ms, _, _ = self.region(legs[n], 1)
            blocks[n] = max(1, int(self.min_s * 1e3 / (ms * self.steps)) + 1)
        out = {n: {"per_round": [], "region_s": [], "windows": []} for n in names}
        for rnd in range(self.rounds):
            k = rnd % len(names)
            for n in names[k:] + names[:k]:
                if self.nvtx:                 # a named range per region, for `ncu --nvtx --nvtx-include <leg>/`
                    self.torch.cuda.nvtx.range_push(n)
                ms, secs, win = self.region(legs[n], blocks[n])
                if self.nvtx:
                    self.torch.cuda.nvtx.range_pop()
                out[n]["per_round"].append(ms)
                out[n]["region_s"].append(secs)
                out[n]["windows"].append(win)
        for n in names:
            r = out[n]
            r["ms_per_step"] = sum(r["per_round"]) / len(r["per_round"])
            r["spread"] = (max(r["per_round"]) - min(r["per_round"])) / r["ms_per_step"]
            r["blocks"] = blocks[n]
        return out


def clock_normalised(flops, ms, sm_mhz, flop_per_clk_sm):
    """Share of the tensor pipe's issue rate at the sampled clock: flops / (148 SM x flop/clk x f x t)."""
    if not sm_mhz:
        return None
    return flops / (148.0 * flop_per_clk_sm * sm_mhz * 1e6 * ms * 1e-3)


def run_ours(args):
    import torch
    from paper_2604_06916_b200 import binding as B
    from paper_2604_06916_b200 import replicas, workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        raise SystemExit(f"bench.py --gpus {args.gpus} needs {args.gpus} ranks but WORLD_SIZE is {world}: launch it as "
                         f"`python -m torch.distributed.run --nnodes=1 --nproc-per-node {args.gpus} --master-addr 127.0.0.1 "
                         f"--master-port <port> bench.py --gpus {args.gpus} ...` (independent replicas, one per GPU)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.lib()
    peaks, peak_src = load_peaks()
    cfg = workloads.CONFIGS[args.workload] if args.workload in workloads.CONFIGS else workloads.config_sweep(
        int(args.workload.split("_g")[-1]))
    layers = cfg.layers
    dev = torch.device("cuda", local_rank)
    warm = max(3, args.warmup)

    def make_data(cfg_):
        acts, data_ = {}, []
        for i, l in enumerate(cfg_.layers):
            X, W, bias = workloads.make_layer(cfg_, i, dev)
            if l.K in acts:
                X = acts[l.K]          # one activation tensor per distinct K (all larger than L2)
            else:
                acts[l.K] = X
            wq, wsf, wts = B.nvfp4_quantize_weight(W)
            Y = torch.empty((l.M, l.N), dtype=torch.bfloat16, device=dev)
            ws = torch.empty(B.linear_workspace_bytes(l.M, l.N, l.K), dtype=torch.uint8, device=dev)
            data_.append(dict(l=l, X=X, W=W, bias=bias, wq=wq, wsf=wsf, wts=wts, Y=Y, ws=ws))
        return data_

    # ---- inputs (resident in HBM), weights quantized once
    data = make_data(cfg)
    torch.cuda.synchronize()

    def fp4_step_of(data_):
        def step():
            for d in data_:
                B.nvfp4_quantize_linear(d["X"], d["wq"], d["wsf"], d["wts"], d["bias"], workspace=d["ws"], out=d["Y"])
        return step

    def bf16_step_of(data_):
        def step():
            for d in data_:
                B.bf16_linear(d["X"], d["W"], d["bias"], out=d["Y"])
        return step

    fp4_step, bf16_step = fp4_step_of(data), bf16_step_of(data)

    # the same FP4 stack with a delayed tensor scale: no amax pass -- the quantizer collects max|x| as a
    # by-product and the scale is rolled forward once per step and layer (one tiny kernel)
    static = []
    for d in data:
        state = torch.zeros(2, dtype=torch.float32, device=dev)
        state[0] = B.sol_amax_bf16(d["X"])[0]
        static.append((d, state))

    def fp4_static_step():
        for d, state in static:
            B.nvfp4_quantize_linear_delayed(d["X"], d["wq"], d["wsf"], d["wts"], d["bias"], state,
                                            workspace=d["ws"], out=d["Y"])
            B.sol_roll_tensor_scale(state)

    # the MXFP4 variant of the stack (32-element blocks, E8M0 scales): no tensor scale, hence no amax pass
    mx = []
    for d in data:
        l = d["l"]
        wq_mx, wsf_mx = B.mxfp4_quantize(d["W"])
        mx.append((d, wq_mx, wsf_mx, torch.empty((l.M, l.K // 2), dtype=torch.uint8, device=dev),
                   torch.empty(B.mxfp4_scale_bytes(l.M, l.K), dtype=torch.uint8, device=dev)))

    def mxfp4_step():
        for d, wq_mx, wsf_mx, xq, xsf in mx:
            B.mxfp4_quantize(d["X"], out=(xq, xsf))
            B.mxfp4_linear(xq, xsf, wq_mx, wsf_mx, d["bias"], out=d["Y"])

    # the FP4 stack through the three separate entries with an event behind every kernel: the split of the
    # step into amax / quantizer / GEMM, taken inside a long loop (same clock state as the step itself)
    split_buf = []
    for d in data:
        l = d["l"]
        split_buf.append((d, torch.empty(1, dtype=torch.float32, device=dev),
                          torch.empty((l.M, l.K // 2), dtype=torch.uint8, device=dev),
                          torch.empty(B.scale_bytes(l.M, l.K), dtype=torch.uint8, device=dev)))
    split_events = []

    def fp4_split_step():
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3 * len(split_buf) + 1)]
        ev[0].record()
        for i, (d, xts, xq, xsf) in enumerate(split_buf):
            B.sol_amax_bf16(d["X"], out=xts)
            ev[3 * i + 1].record()
            B.nvfp4_quantize(d["X"], xts, out=(xq, xsf))
            ev[3 * i + 2].record()
            B.nvfp4_linear(xq, xsf, xts, d["wq"], d["wsf"], d["wts"], d["bias"], out=d["Y"])
            ev[3 * i + 3].record()
        split_events.append(ev)

    gpu_id = str(local_rank)
    try:   # nvidia-smi numbers GPUs its own way: address this one by UUID when it accepts it
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
        if subprocess.run(["nvidia-smi", "-i", uuid, "--query-gpu=uuid", "--format=csv,noheader"], capture_output=True,
                          timeout=20).returncode == 0:
            gpu_id = uuid
    except Exception:
        pass
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
    timer = LegTimer(torch, replicas, dev, dist, sampler, args.steps, args.min_leg_s, args.rounds)
    legs = {"nvfp4": fp4_step, "nvfp4_delayed_scale": fp4_static_step, "mxfp4": mxfp4_step, "bf16": bf16_step}
    res = timer.run(legs, warm)
    B.sol_last_device_status()
    del static, mx

    # ---- split of the step, in one more long region of the instrumented step
    for _ in range(2):
        fp4_split_step()
    torch.cuda.synchronize()
    split_events.clear()
    split_ms, _, split_win = timer.region(fp4_split_step, max(1, int(args.min_leg_s * 1e3 / (res["nvfp4"]["ms_per_step"] * args.steps)) + 1))
    per_layer_split = []
    for i in range(len(split_buf)):
        acc = [0.0, 0.0, 0.0]
        for ev in split_events:
            for j in range(3):
                acc[j] += ev[3 * i + j].elapsed_time(ev[3 * i + j + 1])
        per_layer_split.append([a / len(split_events) for a in acc])
    del split_buf
    split_events.clear()
    B.sol_last_device_status()

    # ---- rollout-scaling sweep point (config 5): the single-stream pair at group size 16, 28 denoising-step
    # calls per sequence, NVFP4 and BF16 sequences in rotated long regions like the legs above
    sweep = None
    if not args.lean and args.sweep_group > 0:
        scfg = workloads.config_sweep(args.sweep_group)
        sdata = make_data(scfg)
        stimer = LegTimer(torch, replicas, dev, dist, sampler, workloads.SWEEP_STEPS, args.min_leg_s, args.rounds)
        sres = stimer.run({"nvfp4": fp4_step_of(sdata), "bf16": bf16_step_of(sdata)}, 2)
        B.sol_last_device_status()
        sflops = flops_of(scfg.layers)
        sweep = {"group": args.sweep_group, "M": scfg.layers[0].M, "calls_per_sequence": workloads.SWEEP_STEPS,
                 "layers": [f"{l.name}:{l.M}x{l.K}->{l.N}" for l in scfg.layers], "res": sres, "flops": sflops}
        del sdata

    # ---- per-kernel durations in isolation: each kernel launched n times back to back between two events on
    # the launching stream.  Every kernel's working set exceeds L2 (X >= 226 MB for the streaming kernels,
    # Y >= 226 MB for the GEMMs); the packed X a GEMM reads is L2-warm, as it is in the step.  These short
    # loops run at burst clocks and are compared with burst peaks; the split above is what adds up to the step.
    per_layer = []
    n_detail = max(5, min(args.steps, 20))
    tot = {"amax": 0.0, "quant": 0.0, "gemm": 0.0}

    def loop_ms(fn):
        fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_detail):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n_detail

    for d, split in zip(data, per_layer_split):
        l = d["l"]
        xts = torch.empty(1, dtype=torch.float32, device=dev)
        xq = torch.empty((l.M, l.K // 2), dtype=torch.uint8, device=dev)
        xsf = torch.empty(B.scale_bytes(l.M, l.K), dtype=torch.uint8, device=dev)
        t_amax = loop_ms(lambda: B.sol_amax_bf16(d["X"], out=xts))
        t_quant = loop_ms(lambda: B.nvfp4_quantize(d["X"], xts, out=(xq, xsf)))
        t_gemm = loop_ms(lambda: B.nvfp4_linear(xq, xsf, xts, d["wq"], d["wsf"], d["wts"], d["bias"], out=d["Y"]))
        t_bf16 = loop_ms(lambda: B.bf16_linear(d["X"], d["W"], d["bias"], out=d["Y"]))
        t_stack = loop_ms(lambda: B.nvfp4_quantize_linear(d["X"], d["wq"], d["wsf"], d["wts"], d["bias"],
                                                           workspace=d["ws"], out=d["Y"]))
        fl = 2.0 * l.M * l.N * l.K
        qbytes = l.M * l.K * 2 + l.M * l.K // 2 + B.scale_bytes(l.M, l.K)
        per_layer.append({
            "layer": l.name, "M": l.M, "K": l.K, "N": l.N,
            "in_step_ms": {"amax": round(split[0], 4), "quant": round(split[1], 4), "gemm": round(split[2], 4)},
            "isolated_ms": {"amax": round(t_amax, 4), "quant": round(t_quant, 4), "gemm": round(t_gemm, 4),
                            "stack": round(t_stack, 4), "bf16": round(t_bf16, 4)},
            "gemm_tflops_in_step": round(fl / split[2] / 1e9, 1), "gemm_tflops_isolated": round(fl / t_gemm / 1e9, 1),
            "bf16_tflops_isolated": round(fl / t_bf16 / 1e9, 1),
            "quant_gbs_in_step": round(qbytes / split[1] / 1e6, 1), "quant_gbs_isolated": round(qbytes / t_quant / 1e6, 1),
            "amax_gbs_in_step": round(l.M * l.K * 2 / split[0] / 1e6, 1),
            "amax_gbs_isolated": round(l.M * l.K * 2 / t_amax / 1e6, 1),
            "stack_speedup_isolated": round(t_bf16 / t_stack, 3),
        })
        tot["amax"] += t_amax
        tot["quant"] += t_quant
        tot["gemm"] += t_gemm
        del xq, xsf
    B.sol_last_device_status()

    flops = flops_of(layers)
    ms_step = res["nvfp4"]["ms_per_step"]
    ms_bf16 = res["bf16"]["ms_per_step"]
    value = world * flops / (ms_step * 1e-3) / 1e12
    bf16_value = world * flops / (ms_bf16 * 1e-3) / 1e12
    quant_bytes = sum(l.M * l.K * 2 + l.M * l.K // 2 + B.scale_bytes(l.M, l.K) for l in layers)
    amax_bytes = sum(l.M * l.K * 2 for l in layers)
    gemm_bytes = sum(l.M * l.K // 2 + B.scale_bytes(l.M, l.K) + l.N * l.K // 2 + B.scale_bytes(l.N, l.K) + 2 * l.N +
                     2 * l.M * l.N for l in layers)
    # split of the step: the instrumented step's shares scaled to the plain step (its events cost a few
    # microseconds each and keep consecutive kernels from overlapping their prologues)
    split_tot = [sum(s[j] for s in per_layer_split) for j in range(3)]
    split_scale = ms_step / sum(split_tot)
    in_step = {"amax_ms": split_tot[0] * split_scale, "quant_ms": split_tot[1] * split_scale,
               "gemm_ms": split_tot[2] * split_scale, "instrumented_step_ms": split_ms, "scale": split_scale}

    # ---- weight refresh after a policy update: merge the rank-32 adapters of every targeted projection
    # and re-quantize it.  FLUX targets to_q/k/v/out: 19 double blocks x 4 + 38 single blocks x 3 = 190
    # matrices of 3072 x 3072.  Timed on 19 distinct matrices (359 MB of base weights, larger than L2)
    # with one merged-weight scratch buffer, as a refresh loop would run it.
    refresh = None
    if world == 1 and not args.lean:
        RN = RK = 3072
        n_mat, n_total = 19, 190
        mats = []
        for i in range(n_mat):
            gen = torch.Generator(device=dev).manual_seed(9000 + i)
            Wm = (torch.randn(RN, RK, generator=gen, device=dev) * RK ** -0.5).to(torch.bfloat16)
            La, Lb = workloads.make_lora(RN, RK, i, dev)
            mats.append((Wm, La, Lb))
        plan = B.LoraRefreshPlan(mats, workloads.LORA_ALPHA / workloads.LORA_RANK)
        refresh_pass = plan.run

        def passes_ms(n):
            refresh_pass()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                refresh_pass()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n

        t_refresh = passes_ms(50) / n_mat
        B.sol_last_device_status()
        fma = RN * RK * workloads.LORA_RANK
        sm_mhz = 1965.0                                    # the part's maximum SM clock
        alu_peak = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12     # FP32 FMA issue: 128 lanes per SM per clock
        refresh = {
            "matrices_per_update": n_total, "shape": [RN, RK], "rank": workloads.LORA_RANK,
            "us_per_matrix": t_refresh * 1e3, "ms_per_update": t_refresh * n_total,
            "elements_per_s": RN * RK / (t_refresh * 1e-3),
            "roofline": {"bound": "alu", "kernel": "lora_merge_kernel", "achieved": 2.0 * fma / (t_refresh * 1e-3) / 1e12,
                         "peak": alu_peak, "unit": "TFLOP/s (fp32)", "frac": 2.0 * fma / (t_refresh * 1e-3) / 1e12 / alu_peak,
                         "traffic": None,
                         "note": "nvfp4_requantize_lora_batch (memset, merge, quantizer per matrix) against the FP32 issue peak "
                                 "148 SM x 128 FMA/clk x 1965 MHz (maximum SM clock); the merge's chain order rules tensor cores out"},
        }
        del mats, plan

    # ---- feed-forward pair with the intermediate kept in NVFP4: MLP-in (GELU) -> MLP-out.  Unfused: two
    # fused-entry calls with a BF16 intermediate (the separate GELU pass such a chain also needs is NOT
    # counted); fused: quantize X, GEMM whose epilogue applies GELU and emits Q(H) with a tensor scale
    # calibrated from the previous call's running amax, GEMM on Q(H).
    mlp_pair = None
    names = [l.name for l in layers]
    if world == 1 and not args.lean and "d_mlp_in" in names and "d_mlp_out" in names:
        d1, d2 = data[names.index("d_mlp_in")], data[names.index("d_mlp_out")]
        l1 = d1["l"]
        xts = torch.empty(1, dtype=torch.float32, device=dev)
        xq = torch.empty((l1.M, l1.K // 2), dtype=torch.uint8, device=dev)
        xsf = torch.empty(B.scale_bytes(l1.M, l1.K), dtype=torch.uint8, device=dev)
        hq = torch.empty((l1.M, l1.N // 2), dtype=torch.uint8, device=dev)
        hsf = torch.empty(B.scale_bytes(l1.M, l1.N), dtype=torch.uint8, device=dev)
        amax = torch.zeros(1, dtype=torch.float32, device=dev)
        t_out = torch.ones(1, dtype=torch.float32, device=dev)
        B.sol_amax_bf16(d1["X"], out=xts)
        B.nvfp4_quantize(d1["X"], xts, out=(xq, xsf))
        B.nvfp4_linear_quantized_out(xq, xsf, xts, d1["wq"], d1["wsf"], d1["wts"], d1["bias"], B.ACT_GELU_TANH, t_out,
                                     amax_out=amax, out=(hq, hsf))
        t_out.copy_(rolled_scale(B, torch, amax))   # calibration from the first call's amax (device to device)

        def pair_unfused():
            B.nvfp4_quantize_linear(d1["X"], d1["wq"], d1["wsf"], d1["wts"], d1["bias"], workspace=d1["ws"], out=d1["Y"])
            B.nvfp4_quantize_linear(d1["Y"], d2["wq"], d2["wsf"], d2["wts"], d2["bias"], workspace=d2["ws"], out=d2["Y"])

        def pair_fused():
            B.sol_amax_bf16(d1["X"], out=xts)
            B.nvfp4_quantize(d1["X"], xts, out=(xq, xsf))
            B.nvfp4_linear_quantized_out(xq, xsf, xts, d1["wq"], d1["wsf"], d1["wts"], d1["bias"], B.ACT_GELU_TANH,
                                         t_out, amax_out=amax, out=(hq, hsf))
            B.nvfp4_linear(hq, hsf, t_out, d2["wq"], d2["wsf"], d2["wts"], d2["bias"], out=d2["Y"])

        t_unf, t_fus = loop_ms(pair_unfused), loop_ms(pair_fused)
        t_unf, t_fus = min(t_unf, loop_ms(pair_unfused)), min(t_fus, loop_ms(pair_fused))
        B.sol_last_device_status()
        pair_flops = 2.0 * l1.M * l1.N * l1.K * 2
        mlp_pair = {"layers": "d_mlp_in (GELU) -> d_mlp_out", "unfused_ms": t_unf, "fused_ms": t_fus,
                    "speedup": t_unf / t_fus, "fused_tflops": pair_flops / t_fus / 1e9,
                    "unfused_tflops": pair_flops / t_unf / 1e9,
                    "note": "unfused = BF16 intermediate, dynamic amax + quantizer per layer, no separate GELU pass "
                            "counted; fused = nvfp4_linear_quantized_out (GELU, calibrated T) feeding nvfp4_linear"}
        del xq, xsf, hq, hsf
        # the same pair in MXFP4 (no amax pass in either form: the format has no tensor scale)
        w1mx, w2mx = B.mxfp4_quantize(d1["W"]), B.mxfp4_quantize(d2["W"])
        xmx = (torch.empty((l1.M, l1.K // 2), dtype=torch.uint8, device=dev),
               torch.empty(B.mxfp4_scale_bytes(l1.M, l1.K), dtype=torch.uint8, device=dev))
        hmx = (torch.empty((l1.M, l1.N // 2), dtype=torch.uint8, device=dev),
               torch.empty(B.mxfp4_scale_bytes(l1.M, l1.N), dtype=torch.uint8, device=dev))

        def mx_unfused():
            B.mxfp4_quantize(d1["X"], B.SF_SWIZZLED_128x4, out=xmx)
            B.mxfp4_linear(xmx[0], xmx[1], w1mx[0], w1mx[1], d1["bias"], out=d1["Y"])
            B.mxfp4_quantize(d1["Y"], B.SF_SWIZZLED_128x4, out=hmx)
            B.mxfp4_linear(hmx[0], hmx[1], w2mx[0], w2mx[1], d2["bias"], out=d2["Y"])

        def mx_fused():
            B.mxfp4_quantize(d1["X"], B.SF_SWIZZLED_128x4, out=xmx)
            B.mxfp4_linear_quantized_out(xmx[0], xmx[1], w1mx[0], w1mx[1], d1["bias"], B.ACT_GELU_TANH, out=hmx)
            B.mxfp4_linear(hmx[0], hmx[1], w2mx[0], w2mx[1], d2["bias"], out=d2["Y"])

        t_mu, t_mf = loop_ms(mx_unfused), loop_ms(mx_fused)
        t_mu, t_mf = min(t_mu, loop_ms(mx_unfused)), min(t_mf, loop_ms(mx_fused))
        B.sol_last_device_status()
        mlp_pair["mxfp4"] = {"unfused_ms": t_mu, "fused_ms": t_mf, "speedup": t_mu / t_mf,
                             "fused_tflops": pair_flops / t_mf / 1e9, "unfused_tflops": pair_flops / t_mu / 1e9,
                             "note": "unfused = BF16 intermediate and a quantizer pass (no GELU pass counted); fused = "
                                     "mxfp4_linear_quantized_out (GELU) feeding mxfp4_linear"}
        del w1mx, w2mx, xmx, hmx

    # ---- single-stream block pair with the concatenated intermediate kept in NVFP4: the first linear's
    # q/k/v columns leave as BF16, its MLP columns pass GELU and are quantized straight into the second
    # linear's input at column 3072; the attention output (a BF16 stand-in of the right shape) is
    # quantized into columns [0, 3072).  Unfused: two fused-entry calls with a BF16 intermediate.
    single_pair = None
    if world == 1 and not args.lean and "s_fused" in names and "s_out" in names:
        d1, d2 = data[names.index("s_fused")], data[names.index("s_out")]
        l1, l2 = d1["l"], d2["l"]
        n_qkv = l1.N - (l2.K - l1.K)          # 21504 - 12288 = 9216 columns feed attention
        attn_w = l2.K - (l1.N - n_qkv)        # 3072 columns of the concat come from attention
        if n_qkv > 0 and n_qkv % 256 == 0 and attn_w == l1.K:
            xts = torch.empty(1, dtype=torch.float32, device=dev)
            xq = torch.empty((l1.M, l1.K // 2), dtype=torch.uint8, device=dev)
            xsf = torch.empty(B.scale_bytes(l1.M, l1.K), dtype=torch.uint8, device=dev)
            cat = (torch.zeros((l1.M, l2.K // 2), dtype=torch.uint8, device=dev),
                   torch.zeros(B.scale_bytes(l1.M, l2.K), dtype=torch.uint8, device=dev))
            y_qkv = torch.empty((l1.M, n_qkv), dtype=torch.bfloat16, device=dev)
            amax = torch.zeros(1, dtype=torch.float32, device=dev)
            t_cat = torch.ones(1, dtype=torch.float32, device=dev)
            attn = d1["X"]                    # stand-in for the attention output: BF16 [M, 3072]

            def single_fused():
                B.sol_amax_bf16(d1["X"], out=xts)
                B.nvfp4_quantize(d1["X"], xts, out=(xq, xsf))
                B.nvfp4_linear_split_out(xq, xsf, xts, d1["wq"], d1["wsf"], d1["wts"], d1["bias"], n_qkv,
                                         B.ACT_GELU_TANH, t_cat, cat, attn_w, y_out=y_qkv, amax_out=amax)
                B.nvfp4_quantize_into(attn, t_cat, cat, 0)
                B.nvfp4_linear(cat[0], cat[1], t_cat, d2["wq"], d2["wsf"], d2["wts"], d2["bias"], out=d2["Y"])

            def single_unfused():
                B.nvfp4_quantize_linear(d1["X"], d1["wq"], d1["wsf"], d1["wts"], d1["bias"], workspace=d1["ws"], out=d1["Y"])
                B.nvfp4_quantize_linear(d2["X"], d2["wq"], d2["wsf"], d2["wts"], d2["bias"], workspace=d2["ws"], out=d2["Y"])

            single_fused()
            # T of the concat: the larger of the two parts' scales (T is monotone in the amax)
            t_cat.copy_(torch.maximum(rolled_scale(B, torch, amax), B.sol_amax_bf16(attn)))
            t_unf, t_fus = loop_ms(single_unfused), loop_ms(single_fused)
            t_unf, t_fus = min(t_unf, loop_ms(single_unfused)), min(t_fus, loop_ms(single_fused))
            B.sol_last_device_status()
            fl2 = 2.0 * l1.M * (l1.N * l1.K + l2.N * l2.K)
            single_pair = {"layers": "s_fused (q/k/v BF16 | GELU(MLP) quantized into the concat) -> s_out",
                           "unfused_ms": t_unf, "fused_ms": t_fus, "speedup": t_unf / t_fus,
                           "fused_tflops": fl2 / t_fus / 1e9, "unfused_tflops": fl2 / t_unf / 1e9,
                           "note": "unfused = BF16 intermediate [M, 15360], dynamic amax + quantizer per layer, no separate "
                                   "GELU or concat pass counted; fused = nvfp4_linear_split_out + nvfp4_quantize_into + "
                                   "nvfp4_linear with a calibrated T"}
            del xq, xsf, cat, y_qkv

    # ---- adaptive layer norm fused with the quantizer (the producer of the q/k/v, MLP-in and single-stream
    # inputs): one pass against torch's layer norm + modulation followed by our amax + quantizer
    ln_quant = None
    if world == 1 and not args.lean:
        l0 = layers[0]
        rps = workloads.SWEEP_TOKENS if l0.M % workloads.SWEEP_TOKENS == 0 else l0.M
        n_s = l0.M // rps
        gen = torch.Generator(device=dev).manual_seed(55)
        sc = (torch.randn(n_s, l0.K, generator=gen, device=dev) * 0.3).to(torch.bfloat16)
        sh = (torch.randn(n_s, l0.K, generator=gen, device=dev) * 0.2).to(torch.bfloat16)
        Xl = data[0]["X"]
        state = torch.ones(1, dtype=torch.float32, device=dev)
        amax = torch.zeros(1, dtype=torch.float32, device=dev)
        lq = (torch.empty((l0.M, l0.K // 2), dtype=torch.uint8, device=dev),
              torch.empty(B.scale_bytes(l0.M, l0.K), dtype=torch.uint8, device=dev))
        B.nvfp4_layernorm_quantize(Xl, sc, sh, rps, state, amax_out=amax, out=lq)
        state.copy_(rolled_scale(B, torch, amax))
        t_fused = loop_ms(lambda: B.nvfp4_layernorm_quantize(Xl, sc, sh, rps, state, amax_out=amax, out=lq))
        xts_l = torch.empty(1, dtype=torch.float32, device=dev)

        def ln_unfused():
            h = torch.nn.functional.layer_norm(Xl, (l0.K,), eps=1e-6)
            h = (h.view(n_s, rps, l0.K) * (1 + sc[:, None, :]) + sh[:, None, :]).view(l0.M, l0.K)
            B.sol_amax_bf16(h, out=xts_l)
            B.nvfp4_quantize(h, xts_l, out=lq)

        t_unf = loop_ms(ln_unfused)
        elems = l0.M * l0.K
        ln_quant = {"shape": [l0.M, l0.K], "fused_us": t_fused * 1e3, "torch_norm_then_amax_quantize_us": t_unf * 1e3,
                    "speedup": t_unf / t_fused, "fused_algorithmic_gbs": elems * 2.5625 / (t_fused * 1e-3) / 1e9,
                    "roofline": {"bound": "hbm", "kernel": "layernorm_quantize_kernel",
                                 "achieved": elems * 2.5625 / (t_fused * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                 "unit": "GB/s", "frac": elems * 2.5625 / (t_fused * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                 "traffic": None, "peak_source": peak_src}}
        del lq, sc, sh

    # ---- BF16 attention of the same block geometry (samples x tokens x hidden / 128 heads), ours and torch's
    attention = None
    if world == 1 and not args.lean and cfg.name.startswith("flux1_12b_g"):
        l0 = cfg.layers[0]
        rps = workloads.SWEEP_TOKENS if l0.M % workloads.SWEEP_TOKENS == 0 else l0.M
        attention = attention_numbers(B, l0.M // rps, rps, l0.K // 128, loop_ms, peaks, peak_src)

    # ---- stage-1 selection and rank metrics at the paper's sizes (48 prompts per epoch, N = 96, K = 24):
    # two launches of one block per prompt, a few microseconds each (launch latency, not throughput)
    selection = None
    if world == 1 and not args.lean:
        gen = torch.Generator(device=dev).manual_seed(123)
        r_ref = torch.randn(48, 96, generator=gen, device=dev)
        r_proxy = (r_ref + 0.25 * torch.randn(48, 96, generator=gen, device=dev)).contiguous()
        seeds = torch.randint(0, 2 ** 62, (48, 96), device=dev, dtype=torch.int64, generator=gen)
        t_sel = loop_ms(lambda: B.solrl_select_contrastive(r_proxy, 24, seeds))
        t_rank = loop_ms(lambda: B.solrl_rank_consistency(r_ref, r_proxy, 4))
        _, m = B.solrl_rank_consistency(r_ref, r_proxy, 4)
        selection = {"prompts": 48, "candidates": 96, "kept": 24, "select_us": t_sel * 1e3, "rank_metrics_us": t_rank * 1e3,
                     "synthetic_mean_tau_rho_top4_bottom4": [round(float(x), 4) for x in m.mean(dim=0).tolist()],
                     "note": "includes the Python binding's output allocation; synthetic proxy = reference + N(0, 0.25^2)"}

    # ---- end to end: pinned HOST activations in, HOST outputs back, copies inside the timed region,
    # through the host-buffer entry point of the C ABI, all six layers per step
    host_x = {}
    e2e_items = []
    h2d = d2h = 0
    for d in ([] if args.lean else data):
        l = d["l"]
        if l.K not in host_x:
            host_x[l.K] = torch.empty((l.M, l.K), dtype=torch.bfloat16).pin_memory()
            host_x[l.K].copy_(d["X"])
        yh = torch.empty((l.M, l.N), dtype=torch.bfloat16).pin_memory()
        e2e_items.append((d, host_x[l.K], yh, torch.empty_like(d["X"])))
        h2d += l.M * l.K * 2
        d2h += l.M * l.N * 2

    # one stream per layer, so that the host-to-device copies queue back to back on their copy engine while
    # the device-to-host copies of earlier layers run on the other (PCIe is full duplex); every layer has
    # its own staging buffers
    side = [torch.cuda.Stream(device=dev) for _ in e2e_items]

    def e2e_step():
        main = torch.cuda.current_stream()
        for st in side:
            st.wait_stream(main)
        for i, (d, xh, yh, xd) in enumerate(e2e_items):
            with torch.cuda.stream(side[i]):
                B.nvfp4_quantize_linear_host(xh, d["wq"], d["wsf"], d["wts"], d["bias"], yh, xd, d["Y"], d["ws"])
        for st in side:
            main.wait_stream(st)

    e2e = None
    if not args.lean:
        e2e_step()
        n_e2e = 3
        ms_e2e, _, _ = LegTimer(torch, replicas, dev, dist, sampler, 1, 0.0, 1).region(e2e_step, n_e2e)
        e2e = {"value": world * flops / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": n_e2e,
               "entry": "nvfp4_quantize_linear_host (pinned host X and Y, copies inside the timed region; "
                        "one stream per layer)"}
    del host_x, e2e_items

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    sampler.stop()

    cpu = None
    if world == 1 and not args.lean:
        cpu = cpu_baseline_on_row_samples(B, torch, workloads, cfg, data, args.cpu_baseline)
        B.sol_last_device_status()

    # ---- clocks: the headline's regions, and every leg's own
    def leg_clocks(r):
        return sampler.window(r["windows"])

    clocks = leg_clocks(res["nvfp4"])
    clocks["per_leg"] = {n: {k: v for k, v in leg_clocks(r).items() if k in ("sm_mhz", "sm_mhz_min", "samples", "reasons", "power_w_max")}
                         for n, r in res.items()}
    split_clk = sampler.window([split_win])
    f_fp4, f_bf16 = clocks["sm_mhz"], clocks["per_leg"]["bf16"]["sm_mhz"]

    def leg_summary(r, fl, flop_clk, clk):
        return {"ms_per_step": round(r["ms_per_step"], 4), "tflops": round(world * fl / r["ms_per_step"] / 1e9, 1),
                "per_round_ms": [round(x, 4) for x in r["per_round"]], "spread": round(r["spread"], 4),
                "blocks_per_region": r["blocks"], "region_s": [round(x, 2) for x in r["region_s"]], "sm_mhz": clk,
                "tensor_issue_util_at_sampled_clock": None if not clk else round(
                    clock_normalised(fl, r["ms_per_step"], clk, flop_clk), 4)}

    legs_out = {n: leg_summary(r, flops, 8192 if n == "bf16" else 32768, clocks["per_leg"][n]["sm_mhz"]) for n, r in res.items()}
    speedup = ms_bf16 / ms_step
    speedup_rounds = [b / a for a, b in zip(res["nvfp4"]["per_round"], res["bf16"]["per_round"])]

    # ---- rooflines.  In-step numbers (taken inside regions of a second or more, power-capped steady state)
    # go against the SUSTAINED measured BF16 peak x 4; isolated 20-launch loops against the BURST peak x 4.
    ratio4 = NOMINAL_FP4_TFLOPS / NOMINAL_BF16_TFLOPS
    gemm_tf_step = flops / (in_step["gemm_ms"] * 1e-3) / 1e12
    gemm_tf_iso = flops / (tot["gemm"] * 1e-3) / 1e12
    peak_sus, peak_burst = peaks["bf16_tflops_sustained"] * ratio4, peaks["bf16_tflops"] * ratio4
    q_gbs_step = quant_bytes / (in_step["quant_ms"] * 1e-3) / 1e9
    q_gbs_iso = quant_bytes / (tot["quant"] * 1e-3) / 1e9
    a_gbs_step = amax_bytes / (in_step["amax_ms"] * 1e-3) / 1e9
    sweep_out = None
    if sweep is not None:
        sr = sweep.pop("res")
        sfl = sweep.pop("flops")
        sclk = {n: sampler.window(r["windows"]) for n, r in sr.items()}
        sweep_out = dict(sweep)
        sweep_out["nvfp4"] = leg_summary(sr["nvfp4"], sfl, 32768, sclk["nvfp4"]["sm_mhz"])
        sweep_out["bf16"] = leg_summary(sr["bf16"], sfl, 8192, sclk["bf16"]["sm_mhz"])
        sweep_out["fp4_over_bf16_speedup"] = round(sr["bf16"]["ms_per_step"] / sr["nvfp4"]["ms_per_step"], 4)
        sweep_out["speedup_per_round"] = [round(b / a, 4) for a, b in zip(sr["nvfp4"]["per_round"], sr["bf16"]["per_round"])]
        sweep_out["reasons"] = sorted(set(sclk["nvfp4"]["reasons"]) | set(sclk["bf16"]["reasons"]))
    g16 = sweep_out["fp4_over_bf16_speedup"] if sweep_out and sweep_out["group"] == 16 else None
    targets = {
        "gemm_pct_of_nominal_9pf": {"value": round(100.0 * gemm_tf_step / NOMINAL_FP4_TFLOPS, 2), "target": 60.0,
                                    "met": gemm_tf_step / NOMINAL_FP4_TFLOPS >= 0.60,
                                    "isolated_burst_loops": round(100.0 * gemm_tf_iso / NOMINAL_FP4_TFLOPS, 2),
                                    "sm_mhz_in_step": split_clk["sm_mhz"],
                                    "note": "9 PF assumes 1965 MHz; under the 1 kW cap the SM clock in the step is the one given"},
        "quantizer_pct_of_8tbs": {"value": round(100.0 * q_gbs_step / NOMINAL_HBM_GBS, 2), "target": 70.0,
                                  "met": q_gbs_step / NOMINAL_HBM_GBS >= 0.70,
                                  "isolated_burst_loops": round(100.0 * q_gbs_iso / NOMINAL_HBM_GBS, 2)},
        "fp4_over_bf16_speedup_g16": {"value": g16, "target": 2.5, "met": None if g16 is None else g16 >= 2.5},
    }
    roofline = {
        "bound": "tensor", "kernel": "gemm_pair_fp4_kernel", "achieved": gemm_tf_step, "peak": peak_sus, "unit": "TFLOP/s",
        "frac": gemm_tf_step / peak_sus, "traffic": int(NCU_TRAFFIC_RATIO["gemm"] * gemm_bytes),
        "traffic_unit": "bytes per step (six launches), d_proj ncu capture scaled by algorithmic bytes",
        "peak_source": f"{peak_src} sustained bf16 {peaks['bf16_tflops_sustained']} TF x 4 (nominal fp4:bf16): the numerator is the "
                       "GEMMs' share of a step timed in regions of >= %.1f s" % args.min_leg_s,
        "isolated": {"achieved": gemm_tf_iso, "peak": peak_burst, "frac": gemm_tf_iso / peak_burst,
                     "peak_source": f"{peak_src} burst bf16 {peaks['bf16_tflops']} TF x 4; 20-launch loops per layer"},
        "step_split_ms": {k: round(v, 4) for k, v in in_step.items()},
        "quantizer": {"bound": "hbm", "kernel": "quantize_kernel", "achieved": q_gbs_step, "peak": peaks["hbm_gbs"],
                      "unit": "GB/s", "frac": q_gbs_step / peaks["hbm_gbs"], "isolated_achieved": q_gbs_iso,
                      "isolated_frac": q_gbs_iso / peaks["hbm_gbs"],
                      "traffic": int(NCU_TRAFFIC_RATIO["quantize"] * quant_bytes), "peak_source": peak_src + " copy bandwidth"},
        "amax": {"bound": "hbm", "kernel": "amax_kernel", "achieved": a_gbs_step, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": a_gbs_step / peaks["hbm_gbs"], "peak_source": peak_src + " copy bandwidth"},
        "targets": targets,
        "fp4_over_bf16_speedup": {"value": round(speedup, 4), "per_round": [round(x, 4) for x in speedup_rounds],
                                  "workload": cfg.name},
        "sweep": sweep_out,
    }

    kernels_per_layer = 3  # amax, quantize (derives and publishes T), GEMM (+1 four-byte memset, not a kernel)
    blocks_fp4 = res["nvfp4"]["blocks"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "nvfp4 (e2m1 x e4m3 block scales, fp32 accumulate, bf16 out)", "data": "synthetic",
        "config": {"workload": cfg.name, "layers": [f"{l.name}:{l.M}x{l.K}->{l.N}" for l in layers],
                   "l2": "smallest activation tensor %.0f MB, tensors touched per step %.0f MB (L2 is 126 MB): %s" % (
                       min(l.M * l.K * 2 for l in layers) / 1e6,
                       sum(l.M * l.K * 2.5625 + l.M * l.N * 2 + l.N * l.K * 0.5625 for l in layers) / 1e6,
                       "every activation tensor is larger than L2" if min(l.M * l.K * 2 for l in layers) > 126e6
                       else "the step's other tensors evict each layer's operands between its uses"),
                   "timing": f"{args.rounds} rounds x {blocks_fp4} blocks of {args.steps} steps per leg: every region >= "
                             f"{args.min_leg_s} s, the rounds start at different legs (nvfp4, delayed scale, mxfp4, bf16); "
                             "ms_per_step is the mean over rounds, max over ranks",
                   "rounds": args.rounds, "blocks_per_region": blocks_fp4,
                   "multi_gpu": "independent replicas, no collective"},
        "pct_of_nominal_fp4_peak": 100.0 * value / world / NOMINAL_FP4_TFLOPS,
        "bf16_stack_tflops": bf16_value, "fp4_over_bf16_speedup": speedup,
        "legs": legs_out,
        "roofline": roofline,
        "weight_refresh": refresh, "mlp_pair_nvfp4_intermediate": mlp_pair, "single_stream_pair_nvfp4_intermediate": single_pair, "layernorm_quantize": ln_quant, "attention_bf16": attention, "stage1_selection": selection,
        "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": kernels_per_layer * len(layers) * args.steps * blocks_fp4 * args.rounds,
        "bf16_vs_torch_matmul_note": "MEASURED_PEAKS bf16 (torch.matmul 8192^3): %.0f burst / %.0f sustained TF" % (
            peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]),
        "per_layer": per_layer,
        # the figures the targets are stated on, last so that they survive a truncated log
        "summary": {"stack_tflops": round(value, 1), "ms_per_step": round(ms_step, 4), "sm_mhz": f_fp4,
                    "gemm_tflops_in_step": round(gemm_tf_step, 1), "gemm_frac_of_sustained_x4": round(gemm_tf_step / peak_sus, 4),
                    "gemm_pct_of_9pf": targets["gemm_pct_of_nominal_9pf"]["value"],
                    "quantizer_gbs_in_step": round(q_gbs_step, 1), "quantizer_pct_of_8tbs": targets["quantizer_pct_of_8tbs"]["value"],
                    "fp4_over_bf16": round(speedup, 3), "bf16_sm_mhz": f_bf16,
                    "sweep_g16_fp4_over_bf16": g16,
                    "targets_met": {k: v["met"] for k, v in targets.items()},
                    "oracle_max_err_over_tol": None if cpu is None else cpu["oracle_max_err_over_tol"]},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_only(args):
    """Small fixed case for profilers: one layer, `steps` passes of the FP4 stack then the BF16 GEMM."""
    import torch
    from paper_2604_06916_b200 import binding as B
    from paper_2604_06916_b200 import workloads

    if args.only == "step":
        # the six-layer step alone (launch lists and profiler captures): warm-up, then `steps` NVFP4 steps and
        # `steps` BF16 steps, each timed as one region
        cfg = workloads.CONFIGS[args.workload]
        M = args.rows if args.rows > 0 else None
        data = []
        for i, l in enumerate(cfg.layers):
            X, W, bias = workloads.make_layer(cfg, i, "cuda", M=M)
            wq, wsf, wts = B.nvfp4_quantize_weight(W)
            Y = torch.empty((X.shape[0], l.N), dtype=torch.bfloat16, device="cuda")
            ws = torch.empty(B.linear_workspace_bytes(X.shape[0], l.N, l.K), dtype=torch.uint8, device="cuda")
            data.append((X, W, bias, wq, wsf, wts, Y, ws))
        res = {}
        for name in ("nvfp4", "bf16"):
            def step():
                for X, W, bias, wq, wsf, wts, Y, ws in data:
                    if name == "nvfp4":
                        B.nvfp4_quantize_linear(X, wq, wsf, wts, bias, workspace=ws, out=Y)
                    else:
                        B.bf16_linear(X, W, bias, out=Y)
            for _ in range(args.warmup):
                step()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                step()
            e1.record()
            torch.cuda.synchronize()
            res[name + "_ms_per_step"] = e0.elapsed_time(e1) / args.steps
        B.sol_last_device_status()
        print(json.dumps({"only": "step", "workload": cfg.name, "rows": data[0][0].shape[0], **res}))
        return
    if args.only == "weight_refresh":
        # eight FLUX attention projections (3072 x 3072, rank-32 adapters) through the batched entry
        n = 3072
        mats = []
        for i in range(8):
            gen = torch.Generator(device="cuda").manual_seed(9000 + i)
            Wm = (torch.randn(n, n, generator=gen, device="cuda") * n ** -0.5).to(torch.bfloat16)
            mats.append((Wm,) + workloads.make_lora(n, n, i, "cuda"))
        plan = B.LoraRefreshPlan(mats, workloads.LORA_ALPHA / workloads.LORA_RANK)
        times = []
        for it in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            plan.run()
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(e0.elapsed_time(e1))
        B.sol_last_device_status()
        print(json.dumps({"only": "weight_refresh", "matrices": 8, "us_per_matrix": 1e3 * sum(times) / len(times) / 8}))
        return
    if args.only.startswith("mxfp4:"):
        # one layer through the MXFP4 quantizer and GEMM
        cfg = workloads.CONFIGS[args.workload]
        index = [l.name for l in cfg.layers].index(args.only.split(":", 1)[1])
        l = cfg.layers[index]
        M = args.rows if args.rows > 0 else l.M
        X, W, bias = workloads.make_layer(cfg, index, "cuda", M=M)
        wq, wsf = B.mxfp4_quantize(W)
        Y = torch.empty((M, l.N), dtype=torch.bfloat16, device="cuda")
        times = []
        for it in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            xq, xsf = B.mxfp4_quantize(X)
            B.mxfp4_linear(xq, xsf, wq, wsf, bias, out=Y)
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(e0.elapsed_time(e1))
        B.sol_last_device_status()
        t = sum(times) / len(times)
        print(json.dumps({"only": args.only, "M": M, "K": l.K, "N": l.N, "mxfp4_stack_ms": t,
                          "mxfp4_stack_tflops": 2.0 * M * l.N * l.K / t / 1e9}))
        return
    if args.only == "single_block":
        # One FLUX-shaped single-stream block forward, NVFP4 against BF16.  The linears, the norm + quantizer
        # and the split / concat epilogues are this library's kernels; attention is torch's scaled-dot-product
        # attention (a library kernel, not part of the path under test) and the gate / residual, BF16 GELU and
        # concat of the BF16 path are plain torch ops.
        import torch.nn.functional as F
        cfg = workloads.CONFIGS[args.workload]
        names = [l.name for l in cfg.layers]
        i1, i2 = names.index("s_fused"), names.index("s_out")
        l1, l2 = cfg.layers[i1], cfg.layers[i2]
        M, H = l1.M, l1.K
        rps = workloads.SWEEP_TOKENS if M % workloads.SWEEP_TOKENS == 0 else M
        n_s, heads, hd = M // rps, H // 128, 128
        n_qkv, n_mlp = 3 * H, l1.N - 3 * H
        X, W1, b1 = workloads.make_layer(cfg, i1, "cuda")
        _, W2, b2 = workloads.make_layer(cfg, i2, "cuda", M=128)
        gen = torch.Generator(device="cuda").manual_seed(77)
        sc, sh, gate = [(torch.randn(n_s, H, generator=gen, device="cuda") * 0.2).to(torch.bfloat16) for _ in range(3)]
        w1q, w2q = B.nvfp4_quantize_weight(W1), B.nvfp4_quantize_weight(W2)
        state = torch.ones(1, dtype=torch.float32, device="cuda")
        amax_in = torch.zeros(1, dtype=torch.float32, device="cuda")
        amax_cat = torch.zeros(1, dtype=torch.float32, device="cuda")
        t_cat = torch.ones(1, dtype=torch.float32, device="cuda")
        xq = (torch.empty((M, H // 2), dtype=torch.uint8, device="cuda"),
              torch.empty(B.scale_bytes(M, H), dtype=torch.uint8, device="cuda"))
        cat = (torch.zeros((M, l2.K // 2), dtype=torch.uint8, device="cuda"),
               torch.zeros(B.scale_bytes(M, l2.K), dtype=torch.uint8, device="cuda"))
        y_qkv = torch.empty((M, n_qkv), dtype=torch.bfloat16, device="cuda")
        y1 = torch.empty((M, l1.N), dtype=torch.bfloat16, device="cuda")
        y2 = torch.empty((M, H), dtype=torch.bfloat16, device="cuda")

        attn_out = torch.empty((M, H), dtype=torch.bfloat16, device="cuda")
        use_ours = {"on": True}

        def attention(qkv):
            if use_ours["on"]:  # this library's kernel reads the fused projection in place and writes [M, H]
                q, k, v = (qkv.view(n_s, rps, -1)[:, :, i * H:(i + 1) * H].unflatten(2, (heads, hd)) for i in range(3))
                B.sol_attention_bf16(q, k, v, out=attn_out.view(n_s, rps, heads, hd))
                return attn_out
            q, k, v = qkv.view(n_s, rps, 3, heads, hd).permute(2, 0, 3, 1, 4)
            o = F.scaled_dot_product_attention(q, k, v)
            return o.transpose(1, 2).reshape(M, H)

        def finish(lin2):
            return X + (gate[:, None, :] * lin2.view(n_s, rps, H)).view(M, H)

        def block_fp4():
            B.nvfp4_layernorm_quantize(X, sc, sh, rps, state, amax_out=amax_in, out=xq)
            B.nvfp4_linear_split_out(xq[0], xq[1], state, *w1q, b1, n_qkv, B.ACT_GELU_TANH, t_cat, cat, H,
                                     y_out=y_qkv, amax_out=amax_cat)
            if use_ours["on"] and use_ours.get("fused", False):
                # attention output quantized in the kernel's epilogue, straight into the concat destination
                q, k, v = (y_qkv.view(n_s, rps, -1)[:, :, i * H:(i + 1) * H].unflatten(2, (heads, hd)) for i in range(3))
                B.sol_attention_nvfp4_out(q, k, v, t_cat, cat, 0)
            else:
                attn = attention(y_qkv)
                B.nvfp4_quantize_into(attn, t_cat, cat, 0)
            B.nvfp4_linear(cat[0], cat[1], t_cat, *w2q, b2, out=y2)
            return finish(y2)

        def block_bf16():
            h = F.layer_norm(X, (H,), eps=1e-6)
            h = (h.view(n_s, rps, H) * (1 + sc[:, None, :]) + sh[:, None, :]).view(M, H)
            B.bf16_linear(h, W1, b1, out=y1)
            attn = attention(y1[:, :n_qkv])
            c = torch.cat((attn, F.gelu(y1[:, n_qkv:], approximate="tanh")), dim=1)
            B.bf16_linear(c, W2, b2, out=y2)
            return finish(y2)

        use_ours["fused"] = False
        out4 = block_fp4()                       # calibrate the delayed scales from the first pass
        state.copy_(rolled_scale(B, torch, amax_in))
        t_cat.copy_(torch.maximum(rolled_scale(B, torch, amax_cat), B.sol_amax_bf16(attention(y_qkv))))
        res = {}
        variants = (("nvfp4", block_fp4, True, False), ("nvfp4_attention_quantized_output", block_fp4, True, True),
                    ("bf16", block_bf16, True, False), ("nvfp4_torch_attention", block_fp4, False, False),
                    ("bf16_torch_attention", block_bf16, False, False))
        # the GPU runs at its power cap and a variant's time depends on what ran before it: every variant is
        # timed in each of three rounds, the rounds start at a different variant, and the mean is reported
        acc = {name: [] for name, *_ in variants}
        for rnd in range(3):
            for name, fn, ours, fused in variants[rnd:] + variants[:rnd]:
                use_ours["on"], use_ours["fused"] = ours, fused
                for _ in range(max(1, args.warmup)):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(args.steps):
                    out = fn()
                e1.record()
                torch.cuda.synchronize()
                acc[name].append(e0.elapsed_time(e1) / args.steps)
                res[name + "_out"] = out
        for name, times in acc.items():
            res[name] = sum(times) / len(times)
        t_attn_by = {}
        for ours in (True, False):
            use_ours["on"] = ours
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                attention(y_qkv)
            e1.record()
            torch.cuda.synchronize()
            t_attn_by[ours] = e0.elapsed_time(e1) / args.steps
        t_attn = t_attn_by[True]
        B.sol_last_device_status()
        diff = (res["nvfp4_out"].float() - res["bf16_out"].float())
        rel = float(diff.pow(2).mean().sqrt() / res["bf16_out"].float().pow(2).mean().sqrt())
        print(json.dumps({"only": "single_block", "M": M, "hidden": H, "nvfp4_ms": res["nvfp4"], "bf16_ms": res["bf16"],
                          "speedup": res["bf16"] / res["nvfp4"], "attention_ms_in_both": t_attn,
                          "attention": "sol_attention_bf16 (this library), then nvfp4_quantize_into",
                          "nvfp4_ms_attention_epilogue_quantizes": res["nvfp4_attention_quantized_output"],
                          "with_torch_attention": {"nvfp4_ms": res["nvfp4_torch_attention"], "bf16_ms": res["bf16_torch_attention"],
                                                   "speedup": res["bf16_torch_attention"] / res["nvfp4_torch_attention"],
                                                   "attention_ms": t_attn_by[False]},
                          "speedup_without_attention": (res["bf16"] - t_attn) / (res["nvfp4"] - t_attn),
                          "rel_rms_difference_of_outputs": rel}))
        return
    if args.only == "attention":
        cfg = workloads.CONFIGS[args.workload]
        l0 = cfg.layers[0]
        rps = workloads.SWEEP_TOKENS if l0.M % workloads.SWEEP_TOKENS == 0 else l0.M
        n_s = args.rows // rps if args.rows > 0 else l0.M // rps
        peaks, peak_src = load_peaks()

        def loop_ms(fn):
            for _ in range(max(1, args.warmup)):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        res = attention_numbers(B, max(1, n_s), rps, l0.K // 128, loop_ms, peaks, peak_src)
        B.sol_last_device_status()
        print(json.dumps({"only": "attention", **res}))
        return
    if args.only == "layernorm_quantize":
        cfg = workloads.CONFIGS[args.workload]
        l0 = cfg.layers[0]
        M = args.rows if args.rows > 0 else l0.M
        X, _, _ = workloads.make_layer(cfg, 0, "cuda", M=M)
        rps = workloads.SWEEP_TOKENS if M % workloads.SWEEP_TOKENS == 0 else M
        gen = torch.Generator(device="cuda").manual_seed(55)
        sc = (torch.randn(M // rps, l0.K, generator=gen, device="cuda") * 0.3).to(torch.bfloat16)
        sh = (torch.randn(M // rps, l0.K, generator=gen, device="cuda") * 0.2).to(torch.bfloat16)
        ts = torch.full((1,), 0.004, dtype=torch.float32, device="cuda")
        times = []
        out = (torch.empty((M, l0.K // 2), dtype=torch.uint8, device="cuda"),
               torch.empty(B.scale_bytes(M, l0.K), dtype=torch.uint8, device="cuda"))
        for it in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.nvfp4_layernorm_quantize(X, sc, sh, rps, ts, out=out)
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(e0.elapsed_time(e1))
        print(json.dumps({"only": "layernorm_quantize", "M": M, "K": l0.K, "us": 1e3 * sum(times) / len(times)}))
        return
    if args.only == "mlp_pair":
        # FLUX feed-forward pair with the intermediate kept in NVFP4 (GELU in the first GEMM's epilogue)
        cfg = workloads.CONFIGS[args.workload]
        names = [l.name for l in cfg.layers]
        i1, i2 = names.index("d_mlp_in"), names.index("d_mlp_out")
        M = args.rows if args.rows > 0 else cfg.layers[i1].M
        X, W1, b1 = workloads.make_layer(cfg, i1, "cuda", M=M)
        _, W2, b2 = workloads.make_layer(cfg, i2, "cuda", M=128)
        w1 = B.nvfp4_quantize_weight(W1)
        w2 = B.nvfp4_quantize_weight(W2)
        xts = B.sol_amax_bf16(X)
        xq, xsf = B.nvfp4_quantize(X, xts)
        t_out = torch.full((1,), 0.01, dtype=torch.float32, device="cuda")
        amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        Y2 = torch.empty((M, W2.shape[0]), dtype=torch.bfloat16, device="cuda")
        times = []
        for it in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            hq, hsf = B.nvfp4_linear_quantized_out(xq, xsf, xts, *w1, b1, B.ACT_GELU_TANH, t_out, amax_out=amax)
            B.nvfp4_linear(hq, hsf, t_out, *w2, b2, out=Y2)
            e1.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(e0.elapsed_time(e1))
        B.sol_last_device_status()
        print(json.dumps({"only": "mlp_pair", "M": M, "ms": sum(times) / len(times)}))
        return
    cfg = workloads.CONFIGS[args.workload]
    index = [l.name for l in cfg.layers].index(args.only)
    l = cfg.layers[index]
    M = args.rows if args.rows > 0 else l.M
    X, W, bias = workloads.make_layer(cfg, index, "cuda", M=M)
    wq, wsf, wts = B.nvfp4_quantize_weight(W)
    Y = torch.empty((M, l.N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.linear_workspace_bytes(M, l.N, l.K), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    times = []
    for it in range(args.warmup + args.steps):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        B.nvfp4_quantize_linear(X, wq, wsf, wts, bias, workspace=ws, out=Y)
        e[1].record()
        B.bf16_linear(X, W, bias, out=Y)
        e[2].record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            times.append((e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])))
    B.sol_last_device_status()
    fl = 2.0 * M * l.N * l.K
    t4 = sum(t[0] for t in times) / len(times)
    t16 = sum(t[1] for t in times) / len(times)
    print(json.dumps({"only": l.name, "M": M, "K": l.K, "N": l.N, "fp4_stack_ms": t4, "bf16_ms": t16,
                      "fp4_stack_tflops": fl / t4 / 1e9, "bf16_tflops": fl / t16 / 1e9}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", default="", help="profile mode: run just this layer of the workload, or 'step' / 'weight_refresh' / 'mlp_pair' / 'mxfp4:<layer>' / 'layernorm_quantize' / 'single_block' / 'attention'")
    ap.add_argument("--rows", type=int, default=0, help="profile mode: override M")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="flux1_12b_g8")
    ap.add_argument("--ref-rows", type=int, default=0, help="rows of the oracle sample (0 = calibrate)")
    ap.add_argument("--rounds", type=int, default=3, help="rotated rounds of the timed legs")
    ap.add_argument("--min-leg-s", type=float, default=1.0, help="minimum length of one timed region in seconds")
    ap.add_argument("--sweep-group", type=int, default=16, help="group size of the rollout-sweep point in the line (0 = none)")
    ap.add_argument("--cpu-baseline", default="workload", choices=["workload", "all"],
                    help="'all' also times the oracle on the row samples of the other configurations and sweep sizes")
    ap.add_argument("--lean", action="store_true",
                    help="sweep mode: skip the end-to-end, weight-refresh and CPU-oracle legs (their keys are null)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.only:
        run_only(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
