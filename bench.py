#!/usr/bin/env python
"""Benchmark of the rotated-MXFP4 linear hot path (rotate -> MXFP4 quantize -> block-scaled FP4
GEMM) at the LLaMA3-8B QKV-projection shape (M=2048 tokens, d=4096, N=6144, bf16 output).

One step = one pass of the whole path over one batch of seeded synthetic activations.  Prints ONE
JSON line (rank 0).  `--impl reference` times the CPU checker (oracle/) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "rotate+MXFP4-quant GB/s and MXFP4 GEMM TFLOP/s, % of roofline (8B shapes)"
WORKLOAD = "llama3_8b_qkv"
N_BUFFER_SETS = 4          # rotated between steps: 4 x ~92 MB of operands > 126 MB of L2


def profiled_traffic(kernel: str, workload: str):
    """DRAM bytes (read + written) per launch of `kernel` on `workload`, from the committed ncu
    summary under profiles/ (a line `dram_bytes_per_launch: N`); None when there is none."""
    import re
    path = os.path.join(ROOT, "profiles", f"{kernel}_{workload}.md")
    if not os.path.exists(path):
        return None
    m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", open(path).read())
    return float(m.group(1)) if m else None


def hold_gpu(stream, ms: float = 5.0):
    """Keeps the stream busy for a few milliseconds BEFORE the first timing event, so that the host
    enqueues the timed launches ahead of the GPU.  Steps of a few tens of microseconds are otherwise
    paced by the Python call overhead rather than by the kernels; the events still measure only
    what lies between them on the device."""
    with torch.cuda.stream(stream):
        torch.cuda._sleep(int(ms * 1e-3 * 1.9e9))


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

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
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(cfg, rows: int, steps: int, warmup: int):
    """The CPU checker, as it stands, on the first `rows` rows of the workload (every stage is
    independent per row).  Weight codes are random: their values do not change the run time."""
    import oracle as O
    from paper_2605_19561_b200 import inputs as I
    xb = I.activations(cfg)[:rows]
    rb, rib, _, _ = I.rotations(cfg)
    wp, wsb = I.random_codes(cfg.N, cfg.d, seed=3)
    wc = O.unpack_codes(wp)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        O.rotated_linear(xb, rb, rib, wc, wsb)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return float(np.mean(times)), cores


REFERENCE_BUDGET_S = 150.0     # wall-clock bound of the whole reference run


def run_reference(args):
    """The oracle, as it stands, timed on the host cores.  One step = one call of the oracle's
    rotated_linear on the first `rows` rows of the workload (every stage is independent per row).
    A call costs about 0.75 s of set-up (decoding R_inter and dequantizing W to float64) plus about
    2.3 ms per row, so the sample per step and, for very large K, the number of steps that fit the
    budget are bounded: the line says what was run."""
    from paper_2605_19561_b200 import inputs as I
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = I.CONFIGS[WORKLOAD]
    steps_req, warmup = max(1, args.steps), min(max(args.warmup, 0), 1)
    per_call_fixed, per_row = 0.9, 0.003
    calls = steps_req + warmup
    rows = int((REFERENCE_BUDGET_S / calls - per_call_fixed) / per_row)
    steps = steps_req
    if rows >= 64:
        rows = min(512, rows)
    else:                                                  # K steps of a meaningful sample do not fit: fewer steps
        rows = 128
        steps = max(1, int(REFERENCE_BUDGET_S / (per_call_fixed + rows * per_row)) - warmup)
    t, cores = time_oracle(cfg, rows, steps, warmup)
    v = rows / t
    sample = (f"first {rows} of {cfg.M} rows per step, all {cfg.d} features and {cfg.N} outputs; {steps} timed steps"
              + ("" if steps == steps_req else f" (of {steps_req} requested: bounded to {REFERENCE_BUDGET_S:.0f} s)"))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "M": cfg.M, "d": cfg.d, "N": cfg.N, "sample": sample},
        "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default: 2000 (the CUDA path), 20 (--impl reference)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD, help="one of inputs.CONFIGS (default: the LLaMA3-8B QKV shape)")
    ap.add_argument("--M", type=int, default=None, help="override the number of tokens (token sweep)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 20 if args.impl == "reference" else 2000
    if args.impl == "reference":
        return run_reference(args)

    from paper_2605_19561_b200 import inputs as I
    from paper_2605_19561_b200 import torq

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    warmup = max(args.warmup, 3)
    cfg = I.CONFIGS[args.workload]
    M, d, N = (args.M or cfg.M), cfg.d, cfg.N
    pk = peaks()

    # ---- inputs (seeded, synthetic; every rank holds its own M rows: weak scaling over tokens)
    xb = I.activations(cfg, M=M)
    # QR of the seeded Gaussian: LAPACK on the host up to d = 4096, on the device above (few host cores)
    rb, rib, _, _ = I.rotations(cfg, device="cpu" if d <= 4096 else "cuda")
    w = I.weights(cfg)
    X0 = I.bf16_bits_to_tensor(xb, "cuda")
    R0, Ri0 = I.bf16_bits_to_tensor(rb, "cuda"), I.bf16_bits_to_tensor(rib, "cuda")
    Wq0, Ws0 = torq.prepare_weights(R0, Ri0, torch.from_numpy(w).cuda())
    # the NVFP4 variant of the same layer (16-element blocks): its own intra rotations and weights
    Ri32_nv = torq.torq_expand_intra16(I.bf16_bits_to_tensor(I.intra_rotations16(cfg), "cuda"))
    torch.cuda.synchronize()
    Wq_nv, Ws_nv, w_ts_nv = torq.prepare_weights_nvfp4(R0, Ri32_nv, torch.from_numpy(w).cuda())
    # activation tensor scale, fixed ahead of time as a calibrated one would be: no rotated element
    # exceeds its token's 2-norm, so the largest norm over the top of the E4M3 range never saturates
    x_ts_nv = float(X0.float().norm(dim=1).max().item()) / (6.0 * 448.0)
    ws_nv = [torch.empty(torq.torq_nvfp4_workspace_bytes(M, d, N), dtype=torch.uint8, device="cuda") for _ in range(2)]
    # the MXINT4 variant (integer codes as E4M3 operand bytes, same rotations as the MXFP4 layer)
    _, W8_i4, Ws_i4 = torq.prepare_weights_mxint4(R0, Ri0, torch.from_numpy(w).cuda())
    ws_i4 = [torch.empty(torq.torq_mxint4_workspace_bytes(M, d, N), dtype=torch.uint8, device="cuda") for _ in range(2)]
    del w
    set_bytes = X0.numel() * 2 + R0.numel() * 2 + Wq0.numel() + M * N * 2
    n_sets = max(2, min(N_BUFFER_SETS, int(8e9 // set_bytes)))     # bounded device memory
    sets = []
    for i in range(n_sets):
        sets.append(dict(X=X0.clone(), R=R0.clone(), Ri=Ri0.clone(), Wq=Wq0.clone(), Ws=Ws0.clone(),
                         Y=torch.empty((M, N), dtype=torch.bfloat16, device="cuda"),
                         ws=torch.empty(torq.torq_workspace_bytes(M, d, N), dtype=torch.uint8, device="cuda")))
    stream = torch.cuda.current_stream()
    fp4_probe = max(torq.torq_probe_fp4_peak(40000) for _ in range(2))     # TFLOP/s, ~1 ms each

    def step(i):
        b = sets[i % n_sets]
        torq.torq_rotated_linear(b["X"], b["R"], b["Ri"], b["Wq"], b["Ws"], Y=b["Y"], workspace=b["ws"])

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    barrier()
    assert torq.torq_last_device_error() == 0

    # ---- timed region: exactly K steps of the whole path, inputs resident in HBM
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = torq.torq_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    hold_gpu(stream)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    launches = torq.torq_launch_count() - launches0
    ms_total = e0.elapsed_time(e1)

    # ---- per-kernel durations: K back-to-back launches of one kernel (operand sets rotated), one
    # event pair around them on the launching stream; average = event time / K.  (With an event
    # between every launch the launch latency that normally overlaps the previous kernel's tail
    # would be charged to the kernel.)
    def codes_scales(b):
        return b["ws"][: M * d // 2].view(M, d // 2), b["ws"][(M * d // 2 + 255) // 256 * 256:][: torq.torq_scales_bytes(M, d)]

    def timed_loop(fn):
        for i in range(3):
            fn(sets[i % n_sets])
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # at most 400 launches per measurement: a kernel shorter than the host's cost of enqueuing it
        # (about 15 us through ctypes) is only timed correctly while the launches queued during the
        # hold last
        k = min(args.steps, 400)
        hold_gpu(stream, ms=10.0)
        a0.record(stream)
        for i in range(k):
            fn(sets[i % n_sets])
        a1.record(stream)
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / k * 1e-3

    def gemm_only(b):
        c, sc = codes_scales(b)
        torq.torq_mxfp4_gemm(c, sc, b["Wq"], b["Ws"], Y=b["Y"])

    def rot_only(b):
        c, sc = codes_scales(b)
        torq.torq_rotate_quantize(b["X"], b["R"], b["Ri"], out_codes=c, out_scales=sc)

    t_gemm = timed_loop(gemm_only)
    # few output tiles: the rotation of the fused call is the split-K pair of kernels, which only runs
    # with the workspace of the fused call; its time is the step minus the GEMM
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    split_k = 2 * ((M + 127) // 128) * ((d + 255) // 256) <= sm_count     # the library's own rule
    t_rot = max(ms_total / args.steps * 1e-3 - t_gemm, 1e-9) if split_k else timed_loop(rot_only)
    # the same activations through the rotation in the paper's own structure (one B x B matrix
    # across blocks, one shared intra-block matrix): reported beside the dense-R_inter path
    t_struct = None
    if d % 256 == 0:
        RB = I.bf16_bits_to_tensor(I.to_bf16_bits(I.orthogonal(d // 32, np.random.Generator(
            np.random.PCG64(I.BASE_SEED + 100 * cfg.cfg_id + 5)))), "cuda")
        Ri1 = Ri0[0].contiguous()

        def struct_only(b):
            c, sc = codes_scales(b)
            torq.torq_rotate_quantize_structured(b["X"], RB, Ri1, out_codes=c, out_scales=sc)

        t_struct = timed_loop(struct_only)

        def struct_layer(b):
            torq.torq_rotated_linear_structured(b["X"], RB, Ri1, b["Wq"], b["Ws"], Y=b["Y"], workspace=b["ws"])

        t_struct_layer = timed_loop(struct_layer)
    # the NVFP4 variant: rotation + quantizer, GEMM, and the whole layer
    def nv_codes_scales(k):
        return (ws_nv[k][: M * d // 2].view(M, d // 2),
                ws_nv[k][(M * d // 2 + 255) // 256 * 256:][: torq.torq_nvfp4_scales_bytes(M, d)])

    nv_i = [0]

    def nv_rot(b):
        nv_i[0] ^= 1
        c, sc = nv_codes_scales(nv_i[0])
        torq.torq_rotate_quantize_nvfp4(b["X"], b["R"], Ri32_nv, x_ts_nv, out_codes=c, out_scales=sc)

    def nv_gemm(b):
        nv_i[0] ^= 1
        c, sc = nv_codes_scales(nv_i[0])
        torq.torq_nvfp4_gemm(c, sc, x_ts_nv, Wq_nv, Ws_nv, w_ts_nv, Y=b["Y"])

    def nv_layer(b):
        nv_i[0] ^= 1
        torq.torq_rotated_linear_nvfp4(b["X"], b["R"], Ri32_nv, x_ts_nv, Wq_nv, Ws_nv, w_ts_nv, Y=b["Y"],
                                       workspace=ws_nv[nv_i[0]])

    t_nv_rot, t_nv_gemm, t_nv_layer = timed_loop(nv_rot), timed_loop(nv_gemm), timed_loop(nv_layer)

    # the MXINT4 variant, likewise
    def i4_bytes_scales(k):
        return ws_i4[k][: M * d].view(M, d), ws_i4[k][(M * d + 255) // 256 * 256:][: torq.torq_scales_bytes(M, d)]

    def i4_rot(b):
        nv_i[0] ^= 1
        c, sc = i4_bytes_scales(nv_i[0])
        torq.torq_rotate_quantize_mxint4(b["X"], b["R"], b["Ri"], out_bytes=c, out_scales=sc)

    def i4_gemm(b):
        nv_i[0] ^= 1
        c, sc = i4_bytes_scales(nv_i[0])
        torq.torq_mxint4_gemm(c, sc, W8_i4, Ws_i4, Y=b["Y"])

    def i4_layer(b):
        nv_i[0] ^= 1
        torq.torq_rotated_linear_mxint4(b["X"], b["R"], b["Ri"], W8_i4, Ws_i4, Y=b["Y"], workspace=ws_i4[nv_i[0]])

    t_i4_rot, t_i4_gemm, t_i4_layer = timed_loop(i4_rot), timed_loop(i4_gemm), timed_loop(i4_layer)
    barrier()
    clocks = sampler.stop()
    assert torq.torq_last_device_error() == 0

    # ---- end to end through the public call with HOST buffers (pinned): every step copies its X
    # host -> device, runs the layer, and copies its Y device -> host, all inside the timed region.
    # Three streams with two device buffers each way: the upload of step i+1 and the download of
    # step i-1 run beside the kernels of step i (PCIe is full duplex), ordered by events.
    Xh = X0.cpu().pin_memory()
    Yh = [torch.empty((M, N), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    e2e_steps = max(3, min(args.steps, 50))
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    Xd = [sets[0]["X"], sets[1]["X"]]
    Yd = [sets[0]["Y"], sets[1]["Y"]]
    wsd = [sets[0]["ws"], sets[1]["ws"]]
    p0 = sets[0]

    def e2e_loop(n):
        x_ready = [torch.cuda.Event() for _ in range(n)]
        y_ready = [torch.cuda.Event() for _ in range(n)]
        x_free = [torch.cuda.Event() for _ in range(n)]
        y_free = [torch.cuda.Event() for _ in range(n)]
        for i in range(n):
            k = i & 1
            with torch.cuda.stream(up):
                if i >= 2:
                    up.wait_event(x_free[i - 2])             # the kernels of step i-2 have read this buffer
                Xd[k].copy_(Xh, non_blocking=True)
                x_ready[i].record(up)
            stream.wait_event(x_ready[i])
            if i >= 2:
                stream.wait_event(y_free[i - 2])             # the download of step i-2 has left this buffer
            torq.torq_rotated_linear(Xd[k], p0["R"], p0["Ri"], p0["Wq"], p0["Ws"], Y=Yd[k], workspace=wsd[k])
            x_free[i].record(stream)
            y_ready[i].record(stream)
            with torch.cuda.stream(down):
                down.wait_event(y_ready[i])
                Yh[k].copy_(Yd[k], non_blocking=True)
                y_free[i].record(down)
        stream.wait_stream(down)
        stream.wait_stream(up)

    e2e_loop(4)
    barrier()
    e0.record(stream)
    e2e_loop(e2e_steps)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1) / e2e_steps
    Yh = Yh[0]

    from paper_2605_19561_b200.sharding import max_over_ranks
    ms_total, ms_e2e, t_rot, t_gemm = max_over_ranks([ms_total, ms_e2e, t_rot, t_gemm], device="cuda")
    ms_step = ms_total / args.steps

    if rank == 0:
        rot_flop = 2.0 * M * d * d + 64.0 * M * d
        rot_bytes = 2.0 * M * d + 2.0 * d * d + 2.0 * 32 * d + M * d / 2 + M * d / 32
        gemm_flop = 2.0 * M * N * d
        gemm_bytes = M * d / 2 + M * d / 32 + N * d / 2 + N * d / 32 + 2.0 * M * N
        # Peak for a kernel timed in a short burst at full clock: the burst figure; when the sampled
        # SM clock sat clearly below its maximum (power cap in a long run): the sustained one.
        at_full_clock = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
                             and clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"])
        bf16_peak = pk["bf16_burst"] if at_full_clock else pk["bf16_sustained"]
        peak_name = f"{pk['source']} bf16 {'burst' if at_full_clock else 'sustained'}"
        # MEASURED_PEAKS.json has no FP4 entry: the denominator is this device's own issue-bound rate of
        # the GEMM's instruction (operands resident in shared memory, no loads), measured just before
        fp4_peak = fp4_probe

        def roof(kernel, t, flop, nbytes, tensor_peak, tensor_name):
            """Roofline record of one kernel: the binding bound is the slower of its HBM and tensor floors."""
            t_hbm, t_tc = nbytes / (pk["hbm_gbs"] * 1e9), flop / (tensor_peak * 1e12)
            if t_tc >= t_hbm:
                ach, peak, unit, bound, src = flop / t / 1e12, tensor_peak, "TFLOP/s", "tensor", tensor_name
            else:
                ach, peak, unit, bound, src = nbytes / t / 1e9, pk["hbm_gbs"], "GB/s", "hbm", f"{pk['source']} HBM copy"
            return {"kernel": kernel, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                    "traffic": profiled_traffic(kernel, args.workload), "peak_source": src,
                    "ms_per_launch": t * 1e3, "algorithmic_flop": flop, "algorithmic_bytes": nbytes}

        pairs = M > 128
        r_rot = roof("rotate_splitk_kernel + splitk_reduce_quantize_kernel" if split_k else
                     ("rotate_quantize_pair_kernel" if pairs else "rotate_quantize_kernel"), t_rot, rot_flop, rot_bytes,
                     bf16_peak, peak_name)
        r_gemm = roof("mxfp4_gemm_pair_kernel" if pairs else "mxfp4_gemm_kernel", t_gemm, gemm_flop, gemm_bytes,
                      fp4_peak, "self-measured: torq_probe_fp4_peak (FP4 block-scaled MMA issue loop, no loads)")
        r_gemm["frac_of_nominal_9000_tflops"] = gemm_flop / t_gemm / 1e12 / 9000.0
        r_gemm["frac_of_4x_measured_bf16"] = gemm_flop / t_gemm / 1e12 / (4.0 * bf16_peak)
        r_rot["frac_of_nominal_2250_tflops"] = rot_flop / t_rot / 1e12 / 2250.0
        dominant, other = (r_rot, r_gemm) if t_rot >= t_gemm else (r_gemm, r_rot)
        out = {
            "metric": METRIC, "value": world * M / (ms_step * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16+mxfp4", "data": "synthetic",
            "config": {"workload": args.workload, "M_per_gpu": M, "d": d, "N": N, "out_dtype": "bf16",
                       "l2": f"{n_sets} operand sets rotated between steps (working set > 126 MB L2)",
                       "sharding": "rows (tokens) per GPU, no collective"},
            "rotate_quant_GBps": rot_bytes / t_rot / 1e9, "rotate_quant_TFLOPs": rot_flop / t_rot / 1e12,
            "gemm_TFLOPs": gemm_flop / t_gemm / 1e12,
            "roofline": dominant, "roofline_other_kernel": other,
            "structured_rotation": None if t_struct is None else (lambda nbytes: {
                "kernel": "rotate_structured_kernel", "what": "rotate+quantize with R_inter = R_B (x) I_32 and one shared "
                "R_intra (the paper's structure, 2d(B+32) flop per token) on the same activations", "bound": "hbm",
                "ms_per_launch": t_struct * 1e3, "achieved": nbytes / t_struct / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": nbytes / t_struct / 1e9 / pk["hbm_gbs"], "algorithmic_bytes": nbytes,
                "traffic": profiled_traffic("rotate_structured_kernel", args.workload),
                "speedup_over_dense_rotation": t_rot / t_struct,
                "whole_layer_ms_per_step": t_struct_layer * 1e3, "whole_layer_tokens_per_s": world * M / t_struct_layer})(
                    2.0 * M * d + 2.0 * (d // 32) ** 2 + 2048.0 + M * d / 2 + M * d / 32),
            "nvfp4_variant": {
                "what": "the same layer in NVFP4 (16-element blocks, E4M3 block scales, float32 tensor scales; "
                        "kind::mxf4nvf4 GEMM), single-pass rotation kernels",
                "rotate_quant_ms": t_nv_rot * 1e3, "rotate_quant_TFLOPs": rot_flop / t_nv_rot / 1e12,
                "rotate_quant_frac": rot_flop / t_nv_rot / 1e12 / bf16_peak,
                "gemm_ms": t_nv_gemm * 1e3, "gemm_TFLOPs": gemm_flop / t_nv_gemm / 1e12,
                "gemm_frac": gemm_flop / t_nv_gemm / 1e12 / fp4_peak,
                "whole_layer_ms_per_step": t_nv_layer * 1e3, "whole_layer_tokens_per_s": world * M / t_nv_layer},
            "mxint4_variant": {
                "what": "the same layer in MXINT4 (32-element blocks, E8M0 scales, integers in [-7,7] fed to the tensor "
                        "cores as E4M3 bytes; kind::mxf8f6f4 GEMM at the 8-bit rate), single-pass rotation kernels",
                "rotate_quant_ms": t_i4_rot * 1e3, "rotate_quant_TFLOPs": rot_flop / t_i4_rot / 1e12,
                "rotate_quant_frac": rot_flop / t_i4_rot / 1e12 / bf16_peak,
                "gemm_ms": t_i4_gemm * 1e3, "gemm_TFLOPs": gemm_flop / t_i4_gemm / 1e12,
                "gemm_frac_of_half_fp4_peak": gemm_flop / t_i4_gemm / 1e12 / (fp4_peak / 2),
                "whole_layer_ms_per_step": t_i4_layer * 1e3, "whole_layer_tokens_per_s": world * M / t_i4_layer},
            "e2e": {"value": world * M / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": Xh.numel() * 2,
                    "d2h_bytes_per_step": Yh.numel() * 2},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if not args.no_cpu_baseline:
            rows = min(512, M)
            t, cores = time_oracle(cfg, rows, 2, 1)
            out["cpu_baseline"] = {"value": rows / t, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                   "sample": f"first {rows} of {M} rows, all features and outputs, 2 timed passes"}
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
