#!/usr/bin/env python
"""Benchmark of the transformed MX-quantized linear layer on B200.

A "step" is one pass of the whole online hot path -- affine transform, MX quantisation, block-scaled
GEMM with the folded bias -- over one batch of synthetic activations, through `latmix_linear`.  The offline
fold + weight quantisation runs once at set-up through `latmix_fold_weights` and is reported separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2_gate_up] [--impl ours|reference]

With N > 1 (launched by torchrun, one rank per GPU) every rank runs the same per-GPU workload on its own rows
(tokens are independent; weights and the transform are replicated; no collective on the data path) and the
job's throughput is the work of all ranks over the slowest rank's time.

`--impl reference` times the CPU oracle (oracle/latmix_oracle.py, as it stands) on a bounded sample of the
same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_17681_b200 import synth  # noqa: E402

FMT_RATIO_TO_BF16 = {"mxfp4": 4.0, "mxfp8": 2.0, "mxint8": 1.0, "mxint4": 2.0, "nvfp4": 4.0}   # nominal dense tensor-rate ratios on B200
METRIC = "fused transform+MX linear throughput"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from an ncu capture of this command
# with the kernel as it is now; None = not captured (or the kernel has changed since the counters were taken).
NCU_DRAM_BYTES_PER_LAUNCH = {"cfg2_gate_up": 219.0e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def pick_regime(clocks, region_ms):
    """Which measured peak a timing belongs with.  "sustained": the power cap was active, or a region long enough to
    be sampled ran with the SM clock well below its maximum; "burst" otherwise (a short region at full clock).  Without
    usable clock samples the burst figure, the larger one, is taken, so that a fraction is never flattered."""
    sm, smax = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if "sw_power_cap" in (clocks.get("reasons") or []):
        return "sustained"
    if sm is None or not smax or region_ms < 100.0:
        return "burst"
    return "sustained" if sm < 0.9 * smax else "burst"


def layer_flops(M, K, N, transform="full"):
    # transform (full K x K matrix on the bf16 pipe, or 32 x 32 blocks on the CUDA cores), block-scaled GEMM (MX pipe)
    return (2.0 * M * K * K if transform == "full" else 64.0 * M * K), 2.0 * M * K * N


def layer_bytes(M, K, N, fmt, transform="full"):
    code = 0.5 if fmt in ("mxfp4", "nvfp4") else 1.0
    scale = 1 / 16.0 if fmt == "nvfp4" else 1 / 32.0
    a_bytes = 2.0 * K * K if transform == "full" else 2.0 * K * 32
    return 2.0 * M * K + a_bytes + N * K * (code + scale) + 4.0 * M * N


def shard_rows(M_total, rank, world):
    """Contiguous row block [lo, hi) of rank `rank` when M_total rows are split over `world` ranks."""
    base, rem = divmod(M_total, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def reduce_max_time(ms, world):
    """Slowest rank's time (the job's time)."""
    if world == 1:
        return ms
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
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
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    power_w_max=max(power) if power else None, samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------------------------------
def oracle_sample_setup(cfg, rows, cols, seed=0):
    """Seeded sample of the workload for the oracle: `rows` activation rows, `cols` output columns."""
    from oracle import latmix_oracle as orc
    layer = synth.make_layer(cfg, device="cpu", M=rows)
    rng = np.random.default_rng(seed)
    col_idx = np.sort(rng.choice(cfg.N, size=min(cols, cfg.N), replace=False))
    X = layer["X"].double().numpy(); A = layer["A"].double().numpy(); b = layer["b"].double().numpy()
    A_inv = layer["A_inv"].double().numpy()
    W = layer["W"].double().numpy()[:, col_idx]; bias = layer["bias"].double().numpy()[col_idx]
    wc, ws, c, _ = orc.fold_weights(A_inv, b, W, bias, cfg.fmt)          # offline, not timed
    return orc, X, A, b, wc, ws, c


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(cfg, rows, cols, steps, warmup):
    orc, X, A, b, wc, ws, c = oracle_sample_setup(cfg, rows, cols)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.latmix_linear(X, A, b, wc, ws, c, cfg.fmt)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    f1, f3 = layer_flops(rows, cfg.K, len(c))
    sec = float(np.mean(times))
    return (f1 + f3) / sec / 1e12, sec


def run_reference(args, cfg, rank, world):
    if rank != 0:
        return
    rows, cols = 1024, 4096
    tflops, sec = time_oracle(cfg, rows, cols, max(1, min(args.steps, 8)), max(0, min(args.warmup, 2)))
    cores = oracle_threads()
    sample = f"{rows} of {cfg.M} rows x {cols} of {cfg.N} output columns per step, full K={cfg.K}; fp64 numpy"
    line = {
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_name(cfg):
    return f"{cfg.name}: X {cfg.M}x{cfg.K} {cfg.x_dtype}, A {cfg.K}x{cfg.K}, W {cfg.K}x{cfg.N}, {cfg.fmt} block {16 if cfg.fmt == 'nvfp4' else 32}"


# ----------------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------------
def run_ours(args, cfg, rank, world, local_rank):
    from paper_2602_17681_b200 import binding as B     # raises if liblatmix.so is missing: no fallback
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    fmt = B.FORMATS[cfg.fmt]
    M, K, N = cfg.M, cfg.K, cfg.N
    peaks = load_peaks()

    # ---- set-up (not timed): inputs on the device, offline fold through the library
    n_sets = 3                                            # rotating sets so that no step finds its data in L2
    layer = synth.make_layer(cfg, device=dev)
    flags = 0
    if args.transform == "blockdiag":
        # the paper's online transform T_3: one orthonormal Hadamard block per MX block, no bias
        blocks, _, A_inv = synth.make_block_transform(K, cfg.seed, "hadamard", a_dtype=cfg.x_dtype, device=dev)
        layer["A"], layer["A_inv"], layer["b"] = blocks, A_inv, torch.zeros(K, dtype=torch.float32, device=dev)
        flags = B.FLAG_BLOCK_DIAG
    g_w = g_a = None
    if cfg.fmt == "nvfp4":
        # the two tensor scales are inputs of the format: calibrated here, at set-up, as max|.| / (448 * 6) of the folded weights
        # and of the transformed activations of the first input set (plain torch products; not part of the timed path)
        g_w = float((layer["A_inv"] @ layer["W"].float()).abs().max()) / (448.0 * 6.0)
        g_a = float((layer["X"].float() @ layer["A"].float() + layer["b"]).abs().max()) * 1.25 / (448.0 * 6.0)
    t0 = time.perf_counter()
    Wq, Wsc, c, _ = B.fold_weights(layer["A_inv"], layer["b"], layer["W"], layer["bias"], fmt, tensor_scale=g_w)
    torch.cuda.synchronize()
    fold_ms = (time.perf_counter() - t0) * 1e3
    sets = []
    for i in range(n_sets):
        X = layer["X"] if i == 0 else synth.make_activations(M, K, cfg.seed + 100 * i + rank, cfg.act, cfg.outlier_frac,
                                                             cfg.outlier_scale, cfg.x_dtype, dev)
        sets.append(dict(X=X, A=layer["A"].clone(), b=layer["b"].clone(), Wq=Wq.clone(), Wsc=Wsc.clone(), c=c.clone(),
                         out=torch.empty(M, N, dtype=torch.float32, device=dev)))
    ws = B.new_workspace(B.OP_LINEAR, M, K, N, fmt, dev)
    if g_a is not None:
        B.workspace_set_tensor_scale(ws, g_a)

    def step(i):
        s = sets[i % n_sets]
        B.linear(s["X"], s["A"], s["b"], s["Wq"], s["Wsc"], s["c"], N, fmt, out=s["out"], ws=ws, flags=flags)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    launches_per_step = None
    if args.graph:
        # the calls only enqueue work on the caller's stream: record one step per input set, replay the recordings
        eager_step, graphs = step, []
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(n_sets):
                g = torch.cuda.CUDAGraph()
                n_before = B.launch_count()
                with torch.cuda.graph(g, stream=side):
                    eager_step(i)
                launches_per_step = B.launch_count() - n_before
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(side)

        def step(i):
            graphs[i % n_sets].replay()
        for i in range(n_sets):
            step(i)
        barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = B.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    launches = B.launch_count() - launches0 if launches_per_step is None else launches_per_step * args.steps
    ms_total = reduce_max_time(ev0.elapsed_time(ev1), world)
    status = B.device_status(ws)
    if status != B.OK:
        raise RuntimeError(f"device status after timed region: {B.status_string(status)}")
    clocks = sampler.stop()
    ms_step = ms_total / args.steps
    f1, f3 = layer_flops(M, K, N, args.transform)
    value = world * (f1 + f3) / (ms_step * 1e-3) / 1e12

    # ---- per-kernel breakdown: the same two kernels, launched through the two half-calls, events around each
    a_codes, a_scales = B.alloc_mx(M, K, fmt, B.SF_TCGEN05, dev)
    if g_a is not None:
        B.set_tensor_scale(a_scales, M, K, fmt, B.SF_TCGEN05, g_a)
    k_iters = max(10, min(args.steps, 200))
    sampler_k = ClockSampler(local_rank)
    sampler_k.start()
    # Each kernel's average launch duration: a batch of back-to-back launches of that kernel alone between two events (the
    # inputs rotate as in the timed region, so no launch finds its operands in L2), as the kernels run inside a step --
    # without the host-side gap an event pair around every single launch would add.
    ek = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for rep in range(2 if k_iters < 100 else 1):         # a short run is repeated so that the clock sampler sees it
        B.quantize_mx(sets[0]["X"], sets[0]["A"], sets[0]["b"], fmt, B.SF_TCGEN05, ws=ws, out=(a_codes, a_scales), flags=flags)
        ek[0].record()
        for i in range(k_iters):
            s = sets[i % n_sets]
            B.quantize_mx(s["X"], s["A"], s["b"], fmt, B.SF_TCGEN05, ws=ws, out=(a_codes, a_scales), flags=flags)
        ek[1].record()
        B.mx_gemm(a_codes, a_scales, sets[0]["Wq"], sets[0]["Wsc"], sets[0]["c"], M, K, N, fmt, out=sets[0]["out"], ws=ws)
        ek[2].record()
        for i in range(k_iters):
            s = sets[i % n_sets]
            B.mx_gemm(a_codes, a_scales, s["Wq"], s["Wsc"], s["c"], M, K, N, fmt, out=s["out"], ws=ws)
        ek[3].record()
        torch.cuda.synchronize()
    clocks_k = sampler_k.stop()
    t_k1 = ek[0].elapsed_time(ek[1]) / k_iters
    t_k2 = ek[2].elapsed_time(ek[3]) / k_iters

    # ---- the tensor pipes' own rate: back-to-back MMAs on operands resident in shared memory, all SMs
    pipe = None
    if not args.no_pipe_probe:
        for kind in ("bf16", "mxf8", "mxf4"):              # first launches carry module loading
            B.tensor_pipe_probe(kind, ws=ws, mma_per_cta=64)
        pipe = {kind: max(B.tensor_pipe_probe(kind, ws=ws) for _ in range(3)) for kind in ("bf16", "mxf8", "mxf4")}

    # Each time is compared with the measured peak of the regime it was taken in: the burst figure when the SM clock sat
    # near its maximum, the sustained one when the power cap held it down; both fractions are printed.
    ratio = FMT_RATIO_TO_BF16[cfg.fmt]
    bf16 = {"burst": peaks["bf16_burst"], "sustained": peaks["bf16_sustained"]}
    regime = pick_regime(clocks, ms_total)
    regime_k = pick_regime(clocks_k, (t_k1 + t_k2) * k_iters * (2 if k_iters < 100 else 1))
    byts = layer_bytes(M, K, N, cfg.fmt, args.transform)
    hbm_s = byts / (peaks["hbm_gbs"] * 1e9)

    def layer_rooflines(p_bf16):
        if args.transform == "full":
            t1_s = f1 / (p_bf16 * 1e12)
        else:   # the block-wise transform is bound by reading X and writing codes and scales
            t1_s = (2.0 * M * K + M * K * ((0.5 if cfg.fmt in ("mxfp4", "nvfp4") else 1.0) + 1 / 32.0)) / (peaks["hbm_gbs"] * 1e9)
        r2 = max(t1_s + f3 / (p_bf16 * ratio * 1e12), hbm_s) * 1e3
        r1 = max((f1 + f3) / (p_bf16 * ratio * 1e12), hbm_s) * 1e3
        return r2, r1
    r2_ms, r1_ms = layer_rooflines(bf16[regime])
    k1_tflops = f1 / (t_k1 * 1e-3) / 1e12
    k2_tflops = f3 / (t_k2 * 1e-3) / 1e12
    p_mx = bf16[regime_k] * ratio
    if M > 128:
        kernel = "bf16_gemm_pair_tc_kernel (MXINT8 expanded to bf16)" if cfg.fmt == "mxint8" else "mx_gemm_wide_tc_kernel (block-scaled GEMM, 256 x 256 CTA-pair tiles)"
    elif cfg.fmt == "mxint8":
        kernel = "mxint8_gemm_decode_i8_tc_kernel (integer MMAs, block scales applied to the int32 sums)" if M <= 64 else "bf16_gemm_pair_tc_kernel (MXINT8 expanded to bf16)"
    else:
        kernel = "mx_gemm_decode_tc_kernel (block-scaled GEMM, operands swapped)" if M <= 64 else "mx_gemm_tc_kernel (block-scaled GEMM)"
    mhz_k = clocks_k.get("sm_mhz")
    roofline = {
        "bound": "tensor", "kernel": kernel,
        "achieved": k2_tflops, "peak": p_mx, "unit": "TFLOP/s", "frac": k2_tflops / p_mx,
        "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(cfg.name),
        "regime": regime_k,
        "peak_source": f"{ratio:g} x bf16 {regime_k} {bf16[regime_k]:g} TFLOP/s of {peaks['source']} (nominal ratio); "
                       f"regime chosen from the SM clock sampled while the kernels were timed",
        "frac_of_burst_peak": k2_tflops / (bf16["burst"] * ratio), "frac_of_sustained_peak": k2_tflops / (bf16["sustained"] * ratio),
        "flops_per_launch": f3, "ms_per_launch": t_k2,
        "cycles_per_launch": t_k2 * 1e-3 * mhz_k * 1e6 if mhz_k else None,
        "clocks_kernels": clocks_k,
        "layer": {"regime": regime, "r2_ms": r2_ms, "r2_frac": r2_ms / ms_step, "r1_ms": r1_ms, "r1_frac": r1_ms / ms_step,
                  "r2_frac_of_burst_peaks": layer_rooflines(bf16["burst"])[0] / ms_step,
                  "r2_frac_of_sustained_peaks": layer_rooflines(bf16["sustained"])[0] / ms_step,
                  "hbm_ms": hbm_s * 1e3, "algorithmic_bytes": byts},
        "kernels": {"transform_quant_ms": t_k1, "transform_quant_tflops": k1_tflops,
                    "transform_quant_frac_of_bf16_peak": k1_tflops / bf16[regime_k],
                    "transform_quant_frac_of_bf16_burst": k1_tflops / bf16["burst"],
                    "mx_gemm_ms": t_k2, "mx_gemm_tflops": k2_tflops},
    }
    if pipe is not None:
        own = {"mxfp4": "mxf4", "nvfp4": "mxf4", "mxfp8": "mxf8", "mxint4": "mxf8", "mxint8": "bf16"}[cfg.fmt]
        roofline["pipe_probe"] = {"tflops": pipe, "frac_of_probe": k2_tflops / pipe[own], "kind": own,
                                  "note": "back-to-back tcgen05.mma 128 x 256 on shared-memory operands, every SM, about 2 ms "
                                          "per kind, at the clock the probe itself ran at"}
    if M <= 64:
        # small batches: the dominant kernel streams the weights once; algorithmic bytes = codes + scales of both operands + result
        code = 0.5 if cfg.fmt in ("mxfp4", "nvfp4") else 1.0
        k2_bytes = (N + M) * K * (code + 1 / 32.0) + 4.0 * M * N
        gbs = k2_bytes / (t_k2 * 1e-3) / 1e9
        roofline.update({"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "peak_source": f"copy bandwidth of {peaks['source']}", "bytes_per_launch": k2_bytes})
        for key in ("frac_of_burst_peak", "frac_of_sustained_peak", "flops_per_launch", "pipe_probe"):
            roofline.pop(key, None)

    # ---- end to end through the public call with HOST buffers (pinned), copies inside the timed region
    e2e = None
    cpu_baseline = None
    if rank == 0 or world > 1:
        # Two slots, each with its own stream, device buffers, workspace and pinned result buffer: while one step's
        # result travels back over PCIe the next step's input is copied in and computed.  Every step still copies its
        # own input in and its own result out.
        hX = torch.empty(M, K, dtype=sets[0]["X"].dtype).pin_memory()
        hX.copy_(sets[0]["X"].cpu())
        slots = []
        for i in range(2):
            slots.append(dict(stream=torch.cuda.Stream(device=dev), dX=torch.empty_like(sets[0]["X"]),
                              dout=sets[i]["out"], hout=torch.empty(M, N, dtype=torch.float32).pin_memory(),
                              ws=ws if i == 0 else B.new_workspace(B.OP_LINEAR, M, K, N, fmt, dev)))
            if g_a is not None:
                B.workspace_set_tensor_scale(slots[-1]["ws"], g_a)
        torch.cuda.synchronize()
        n_e2e = max(4, min(args.steps, 10))

        def e2e_step(i):
            sl = slots[i % 2]
            with torch.cuda.stream(sl["stream"]):
                sl["dX"].copy_(hX, non_blocking=True)
                B.linear(sl["dX"], sets[0]["A"], sets[0]["b"], sets[0]["Wq"], sets[0]["Wsc"], sets[0]["c"], N, fmt,
                         out=sl["dout"], ws=sl["ws"], flags=flags)
                sl["hout"].copy_(sl["dout"], non_blocking=True)

        def join_slots():
            for sl in slots:
                torch.cuda.current_stream().wait_stream(sl["stream"])

        def fork_slots():
            for sl in slots:
                sl["stream"].wait_stream(torch.cuda.current_stream())
        e2e_step(0); e2e_step(1)
        join_slots()
        barrier()
        ev0.record()
        fork_slots()
        for i in range(n_e2e):
            e2e_step(i)
        join_slots()
        ev1.record()
        barrier()
        for sl in slots:
            if B.device_status(sl["ws"]) != B.OK:
                raise RuntimeError("device status after the end-to-end region")
        hout = slots[0]["hout"]
        ms_e2e = reduce_max_time(ev0.elapsed_time(ev1), world) / n_e2e
        e2e = {"value": world * (f1 + f3) / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": hX.numel() * hX.element_size(), "d2h_bytes_per_step": hout.numel() * 4}

    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.transform == "full" and cfg.fmt != "nvfp4":
        rows, cols = 1024, 4096
        tf, sec = time_oracle(cfg, rows, cols, steps=5, warmup=1)
        cpu_baseline = {"value": tf, "unit": "TFLOP/s", "cores": oracle_threads(), "kind": "oracle",
                        "sample": f"{rows} of {M} rows x {cols} of {N} output columns, full K={K}, 5 timed passes of {sec:.2f} s",
                        "sec_per_pass": sec}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"mxfp4": "fp4(e2m1)+e8m0 x bf16 transform", "mxfp8": "fp8(e4m3)+e8m0 x bf16 transform",
                      "mxint8": "int8+e8m0 x bf16 transform", "mxint4": "int4 (as e4m3 bytes)+e8m0 x bf16 transform",
                      "nvfp4": "fp4(e2m1)+e4m3 per 16+fp32 tensor scale x bf16 transform"}[cfg.fmt],
            "data": "synthetic",
            "config": {"workload": workload_name(cfg) + (", online transform: 32x32 Hadamard blocks (T3)" if args.transform == "blockdiag" else ""),
                       "rows_per_gpu": M, "parallelism": f"rows x{world} (replicated weights, no collective)",
                       "l2": f"{n_sets} rotating input/weight/output sets of {byts / 1e6:.0f} MB each (> 126 MB L2)",
                       "launch": "CUDA graph replay" if args.graph else "stream launches",
                       "fold_ms_offline": fold_ms},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------------
# Offline folds (not the headline: --op fold / --op fold_two_sided time the weight-side preparation)
# ----------------------------------------------------------------------------------------------------
def run_fold(args, cfg, local_rank):
    from paper_2602_17681_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    fmt = B.FORMATS[cfg.fmt]
    K, N = cfg.K, cfg.N
    peaks = load_peaks()
    layer = synth.make_layer(cfg, device=dev, M=32)
    two = args.op == "fold_two_sided"
    if args.op == "mse":
        M = cfg.M
        X = synth.make_activations(M, K, cfg.seed, cfg.act, cfg.outlier_frac, cfg.outlier_scale, cfg.x_dtype, dev)
        mse_flags = 0
        if args.mse_transform == "identity":
            A = A_inv = b_t = None
        elif args.mse_transform == "hadamard":
            A, b_t, A_inv = synth.make_block_transform(K, cfg.seed, "hadamard", a_dtype=cfg.x_dtype, device=dev)
            mse_flags = B.FLAG_BLOCK_DIAG
        else:
            A, b_t, A_inv = synth.make_transform(K, cfg.seed, cfg.x_dtype, cfg.b_std, dev)
        ws = B.new_workspace(B.OP_TRANSFORMATION_MSE, M, K, 0, fmt, dev)
        mse_out = {}

        def call():
            mse_out["mse"], mse_out["blk"] = B.transformation_mse(X, A, b_t, A_inv, fmt, ws=ws, flags=mse_flags, block=args.block)
        n_prod = {"identity": 0, "hadamard": 1, "full": 2}[args.mse_transform]
        flops = 2.0 * M * K * K * n_prod                         # the transform and the back-mapping product
        issued = 2.0 * M * K * K * ({"identity": 0, "hadamard": 9, "full": 1 + 9}[args.mse_transform])   # back-mapping: three bf16 terms per operand
    elif two:
        A_out, v_out, _ = synth.make_transform(N, cfg.seed + 1, "f32", device=dev)
        ws = B.new_workspace(B.OP_FOLD_TWO_SIDED, 0, K, N, fmt, dev)
        call = lambda: B.fold_weights_two_sided(layer["A_inv"], layer["b"], layer["W"], layer["bias"], A_out, v_out, fmt, ws=ws)
        flops = 2.0 * K * K * N + 2.0 * K * N * N
        issued = 9 * 2.0 * K * K * N + 3 * 2.0 * K * N * N       # three-term operands: 3 x 3 and 1 x 3 bf16 products
    else:
        f32w = args.weights == "f32"
        W = layer["W"].float() if f32w else layer["W"]
        # fp32 weights reach the tensor cores with room for their three bf16 terms in the workspace
        ws = torch.zeros(B.workspace_bytes(B.OP_FOLD_WEIGHTS, 0, K, N, fmt) + (6 * K * N if f32w else 0), dtype=torch.uint8, device=dev)
        call = lambda: B.fold_weights(layer["A_inv"], layer["b"], W, layer["bias"], fmt, ws=ws)
        flops = 2.0 * K * K * N
        issued = (9 if f32w else 3) * flops
    steps, warmup = min(args.steps, 50), max(3, min(args.warmup, 5))
    for _ in range(warmup):
        call()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    n0 = B.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        call()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / steps
    if B.device_status(ws) != B.OK:
        raise RuntimeError("device status after timed region")
    regime = pick_regime(clocks, ms * steps)
    peak = peaks["bf16_" + regime]
    print(json.dumps({
        "metric": "transformation MSE diagnostic time" if args.op == "mse" else "offline fold + weight quantisation time", "value": ms, "unit": "ms", "n_gpus": 1, "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 x 3-term bf16 -> f32", "data": "synthetic",
        "config": dict({"workload": workload_name(cfg), "op": args.op, "weights": args.weights, "algorithmic_gflop": flops / 1e9,
                        "issued_bf16_gflop": issued / 1e9, "l2": "operands larger than L2"},
                       **({"block": args.block, "transform": args.mse_transform, "transformation_mse": float(mse_out["mse"]),
                           "block_err_min_max": [float(mse_out["blk"].min()), float(mse_out["blk"].max())]} if args.op == "mse" else {})),
        "clocks": clocks, "gpu_launches": int(B.launch_count() - n0),
        "roofline": {"bound": "tensor", "achieved": issued / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                     "frac": issued / (ms * 1e-3) / 1e12 / peak, "traffic": None,
                     "regime": regime,
                     "note": "issued bf16 flops (three-term splits) of all kernels of the call over the bf16 %s %s peak; "
                             "algorithmic rate %.1f TFLOP/s" % (peaks["source"], regime, flops / (ms * 1e-3) / 1e12)},
    }), flush=True)


# ----------------------------------------------------------------------------------------------------
# Standalone quantiser (--op quantize): Eq. "q_mx" on the workload's activations, no transform -- memory-bound
# ----------------------------------------------------------------------------------------------------
def run_quantize(args, cfg, local_rank):
    from paper_2602_17681_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    fmt = B.FORMATS[cfg.fmt]
    M, K = cfg.M, cfg.K
    peaks = load_peaks()
    in_bytes = 2 if cfg.x_dtype == "bf16" else 4
    byts = M * K * (in_bytes + (0.5 if cfg.fmt == "mxfp4" else 1.0) + 1 / 32.0)
    n_sets = max(3, int(3 * 126e6 / byts) + 1)              # rotating sets: no step finds its input in L2
    Xs = [synth.make_activations(M, K, cfg.seed + i, cfg.act, cfg.outlier_frac, cfg.outlier_scale, cfg.x_dtype, dev) for i in range(n_sets)]
    outs = [B.alloc_mx(M, K, fmt, B.SF_TCGEN05, dev) for _ in range(n_sets)]
    ws = B.new_workspace(B.OP_QUANTIZE_MX, M, K, 0, fmt, dev)
    steps, warmup = min(args.steps, 2000), max(3, min(args.warmup, 20))
    for i in range(warmup):
        B.quantize_mx(Xs[i % n_sets], None, None, fmt, ws=ws, out=outs[i % n_sets])
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    n0 = B.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(steps):
        B.quantize_mx(Xs[i % n_sets], None, None, fmt, ws=ws, out=outs[i % n_sets])
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / steps
    if B.device_status(ws) != B.OK:
        raise RuntimeError("device status after timed region")
    gbs = byts / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "standalone MX quantiser bandwidth", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": f"{cfg.x_dtype} -> {cfg.fmt}", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: X {M}x{K} {cfg.x_dtype} -> {cfg.fmt} block 32, tiled scale layout", "op": args.op,
                   "algorithmic_bytes": byts, "l2": f"{n_sets} rotating input/output sets"},
        "clocks": clocks, "gpu_launches": int(B.launch_count() - n0),
        "roofline": {"bound": "hbm", "kernel": "quantize_rows_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                     "note": "input read once + codes + scale bytes over the copy bandwidth of %s" % peaks["source"]},
    }), flush=True)


# ----------------------------------------------------------------------------------------------------
# Tensor-pipe issue-rate probe (--op mma_peak): what the pipes deliver when nothing but MMAs runs
# ----------------------------------------------------------------------------------------------------
def run_mma_peak(args, local_rank):
    from paper_2602_17681_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    ws = B.new_workspace(B.OP_QUANTIZE_MX, 0, 64, 0, B.MXFP4, dev)
    nominal = {"bf16": 1.0, "mxf8": 2.0, "mxf4": 4.0, "nvf4": 4.0, "mxf4_pair": 4.0}
    for kind in nominal:                                   # warm-up
        B.tensor_pipe_probe(kind, ws=ws)
    sampler = ClockSampler(local_rank)
    sampler.start()
    n0 = B.launch_count()
    reps = max(3, min(args.steps, 50))
    out = {k: max(B.tensor_pipe_probe(k, ws=ws) for _ in range(reps)) for k in nominal}
    long_run = {k: B.tensor_pipe_probe(k, ws=ws, mma_per_cta=1 << 22) for k in ("bf16", "mxf4")}   # about 0.3 s each
    clocks = sampler.stop()
    print(json.dumps({
        "metric": "tensor pipe issue rate", "value": out["mxf4"], "unit": "TFLOP/s", "n_gpus": 1, "steps": reps, "warmup": 1,
        "higher_is_better": True, "vs_baseline": None, "dtype": "mxf4 / mxf8f6f4 / bf16 / mxf4nvf4", "data": "synthetic",
        "config": {"workload": "back-to-back tcgen05.mma 128 x 256 x (16 | 32 | 64), operands resident in shared memory, "
                               "one CTA per SM, best of %d launches of about 2 ms" % reps, "op": args.op},
        "clocks": clocks, "gpu_launches": int(B.launch_count() - n0),
        "tflops": out, "tflops_long_run": long_run,
        "ratio_to_bf16_probe": {k: out[k] / out["bf16"] for k in out},
        "measured_cublas_bf16": {"burst": peaks["bf16_burst"], "sustained": peaks["bf16_sustained"], "source": peaks["source"]},
        "nominal_ratio_to_bf16": nominal,
    }), flush=True)


def spawn_ranks(args):
    """`bench.py --gpus N` without a launcher: start N ranks of this same command under torch.distributed.run (one per
    GPU, rendezvous on 127.0.0.1) and return its exit code.  Refuses when fewer than N GPUs are visible."""
    if not args.plumbing_only and args.impl == "ours":
        have = torch.cuda.device_count()
        if have < args.gpus:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} asked for but {have} GPU(s) visible; not running on fewer\n")
            return 2
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_plumbing(args, rank, world):
    """The multi-rank plumbing without a GPU: rendezvous on gloo, barrier, row shards, max-over-ranks of a per-rank time."""
    import torch.distributed as dist
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
        dist.barrier()
    lo, hi = shard_rows(synth.CONFIGS[args.workload].M * world, rank, world)
    ms = reduce_max_time(1.0 + rank, world)
    rows = torch.tensor([hi - lo], dtype=torch.int64)
    if world > 1:
        dist.all_reduce(rows)
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"plumbing_only": True, "n_gpus": world, "ms_slowest_rank": ms, "rows_total": int(rows.item())}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_gate_up", choices=sorted(synth.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-pipe-probe", action="store_true", help="skip the tensor-pipe issue-rate probe")
    ap.add_argument("--graph", action="store_true", help="record each step in a CUDA graph and time the replays (small batches are launch-bound)")
    ap.add_argument("--transform", default="full", choices=["full", "blockdiag"],
                    help="full K x K learned-style matrix (the configuration the metric is quoted on) or the paper's online "
                         "block transform T3 (32 x 32 Hadamard blocks)")
    ap.add_argument("--weights", default="bf16", choices=["bf16", "f32"], help="--op fold: dtype of the unfolded weights")
    ap.add_argument("--op", default="layer", choices=["layer", "fold", "fold_two_sided", "mse", "quantize", "mma_peak"],
                    help="layer: the online path (the metric); fold / fold_two_sided: time the offline weight preparation; "
                         "mse: the transformation-MSE diagnostic (time and values); quantize: the standalone quantiser (no "
                         "transform); mma_peak: issue-rate probe of the tensor pipes")
    ap.add_argument("--plumbing-only", action="store_true",
                    help="no GPU work: run only the launch, rendezvous (gloo), barrier and max-over-ranks plumbing of --gpus N")
    ap.add_argument("--block", type=int, default=32, help="--op mse: block size B of the quantiser (8, 16, 32, 64 or 128)")
    ap.add_argument("--mse-transform", default="full", choices=["identity", "full", "hadamard"],
                    help="--op mse: no transform, the full learned-style matrix, or 32 x 32 Hadamard blocks")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = synth.CONFIGS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)\n")
        sys.exit(2)
    if args.plumbing_only:
        run_plumbing(args, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return
    if args.op == "mma_peak":
        if rank == 0:
            run_mma_peak(args, local_rank)
        return
    if args.op != "layer":
        if rank == 0:
            (run_quantize if args.op == "quantize" else run_fold)(args, cfg, local_rank)
        return
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if torch.cuda.device_count() < world:
            sys.stderr.write(f"bench.py: {world} ranks but only {torch.cuda.device_count()} GPU(s) visible\n")
            sys.exit(2)
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, cfg, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
