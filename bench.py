#!/usr/bin/env python
"""Benchmark of the MixLoRA FFN block (forward + aux loss + backward) on B200.

    python bench.py --gpus N --steps K --warmup W          # the CUDA library
    python bench.py --impl reference ...                   # the CPU oracle, bounded sample per step

One "step" is one pass of the whole hot path over one synthetic batch of the LLaMA-2-7B
shaped workload (8192 tokens per GPU, 8 experts, top-2, rank 16): forward, auxiliary loss,
backward with LoRA, router and input gradients.  Rank 0 prints one JSON line.
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

from paper_2404_15159_b200 import synth

METRIC = "mixlora_ffn_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
AUX_COEF = 0.01


def workload_by_name(name: str) -> synth.Workload:
    table = {"c1": synth.c1, "c2": synth.c2, "c3": synth.c3, "c4": synth.c4, "llama3-8b": synth.llama3_8b,
             "wide-2b": synth.wide_2b}
    if name in table:
        return table[name]()
    if name.startswith("c5:"):                      # c5:N,k,r,T
        n, k, r, t = (int(v) for v in name[3:].split(","))
        return synth.c5(n, k, r, t)
    raise SystemExit(f"unknown workload {name}")


# ----------------------------------------------------------------------------------------
# flop / byte model of the stages (algorithmic, per step)
# ----------------------------------------------------------------------------------------
def stage_flops(w: synth.Workload, want_dx: bool) -> dict:
    T, d, f, N, k, r = w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank
    U = 2.0 * T * d * f
    Nr = N * r
    NP = (N + 7) // 8 * 8
    fl = {
        "gemm_gate_up": 2 * U + 2 * 2.0 * T * d * Nr,          # W1, W3 once per token + LoRA-A of every expert
        "gemm_down": U + 2.0 * T * Nr * d,                     # W2 on the gate-weighted sum + LoRA-B down
        "gemm_dgrad_down": U + 2.0 * T * d * Nr,               # dy W2 + B_d^T dy
        "gemm_dx": (2 * U + 2 * 2.0 * T * Nr * d + 2.0 * T * NP * d) if want_dx else 0.0,
    }
    return fl


def load_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------
# clocks sampler
# ----------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        rows = [s for s in self.samples if t0 <= s[0] <= t1 + 0.1] or self.samples
        for _, line in rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------
# CPU oracle leg
# ----------------------------------------------------------------------------------------
def oracle_sample(w: synth.Workload, tensors: dict, sample_tokens: int, want_dx: bool):
    """One oracle forward + aux + backward on the first `sample_tokens` tokens.  Returns seconds."""
    from oracle import mixlora_oracle as orc
    xs, dys = tensors["x"][:sample_tokens], tensors["dy"][:sample_tokens]
    params = synth.params_of(tensors)
    t0 = time.perf_counter()
    y, saved = orc.ffn_forward(xs, params, w.top_k, w.lora_alpha)
    orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], AUX_COEF)
    orc.ffn_backward(xs, params, dys, saved, aux_coef=AUX_COEF, want_dx=want_dx)
    return time.perf_counter() - t0


def threads_used() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload_by_name(args.workload)
    sample = args.ref_sample
    if sample <= 0:
        # size the per-step sample so that the whole run (warm-up + timed steps) takes about two minutes: one
        # calibration pass over 64 tokens gives the oracle's time per token on this host
        probe = synth.generate(w.with_(tokens=64))
        per_token = oracle_sample(w, probe, 64, True) / 64
        sample = int(120.0 / ((args.warmup + args.steps) * per_token))
        sample = max(16, min(256, sample))
    tensors = synth.generate(w.with_(tokens=sample))
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_sample(w, tensors, sample, True)
        if i >= args.warmup:
            times.append(dt)
    per_step = float(np.mean(times))
    value = sample / per_step
    cores = threads_used()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "tokens_per_gpu": w.tokens, "d_model": w.d_model, "d_ff": w.d_ff,
                   "n_experts": w.n_experts, "top_k": w.top_k, "rank": w.rank},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} tokens of the workload per step, full d_model/d_ff, forward + aux + "
                                   f"backward with dx, float64 numpy"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------
# CUDA leg
# ----------------------------------------------------------------------------------------
def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2404_15159_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local)
    use_dist = world > 1 or args.force_dist
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    elif use_dist:      # one rank going through the collective path (checks the stream and event plumbing on one GPU)
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29541", rank=0, world_size=1,
                                device_id=torch.device("cuda", local))

    w = workload_by_name(args.workload)
    want_dx = not args.no_dx
    bf16 = w.dtype == "bf16"
    act = torch.bfloat16 if bf16 else torch.float32
    # every rank holds the same weights and its own batch of tokens (data parallel, weak scaling)
    tensors = synth.generate(w.with_(seed=w.seed))
    if rank > 0:
        rng = np.random.Generator(np.random.Philox(key=w.seed + 1000 + rank))
        tensors["x"] = synth.round_to_bf16(rng.standard_normal(tensors["x"].shape, dtype=np.float32))
        tensors["dy"] = synth.round_to_bf16(rng.standard_normal(tensors["dy"].shape, dtype=np.float32))
    dev = {}
    for n, v in tensors.items():
        if v is None:
            dev[n] = None
        elif n in ("w_router", "router_bias"):
            dev[n] = torch.from_numpy(v).cuda()
        else:
            dev[n] = torch.from_numpy(v).cuda().to(act)
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                         B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, True)
    y = torch.empty(w.tokens, w.d_model, dtype=act, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    from paper_2404_15159_b200 import dp
    offsets, total = dp.flat_grad_layout(w.d_model, w.d_ff, w.n_experts, w.rank)
    flat = torch.zeros(total, dtype=torch.float32, device="cuda")        # one buffer => one all-reduce
    g = {n: flat[off:off + size] for n, (off, size) in offsets.items()}
    if want_dx:
        g["d_x"] = torch.empty(w.tokens, w.d_model, dtype=act, device="cuda")
    grads = B.make_grads(accumulate=0, **g)

    def step():
        B.mixlora_ffn_forward(shape, params, y, ws)
        B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
        B.mixlora_ffn_backward(shape, params, dev["dy"], AUX_COEF, ws, grads)

    if use_dist:
        # data-parallel sum of the LoRA and router gradients (one flat buffer, one NCCL all-reduce) on a second
        # stream: it starts when the parameter gradients are enqueued and runs beside the input-gradient product
        comm = torch.cuda.Stream()
        ev_ready = torch.cuda.Event()
        ev_ready.record()

        def step():                        # noqa: F811
            B.mixlora_ffn_forward(shape, params, y, ws)
            B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
            B.mixlora_ffn_backward_overlap(shape, params, dev["dy"], AUX_COEF, ws, grads, ev_ready)
            comm.wait_event(ev_ready)
            with torch.cuda.stream(comm):
                dist.all_reduce(flat)
            torch.cuda.current_stream().wait_stream(comm)

    M = max(1, args.models)
    if M > 1:
        # Multi-model variant (Section 3.3 (II)): the batch is split over M adapters that share the frozen FFN and
        # go through one multi-model call; each adapter has its own workspace, outputs and gradient buffers (the
        # LoRA / router tensors are re-used between adapters here, which does not change the work).
        Tm = w.tokens // M
        m_shapes, m_params, m_ys, m_ws, m_dys, m_grads, m_keep = [], [], [], [], [], [], []
        for m in range(M):
            sl = slice(m * Tm, (m + 1) * Tm)
            sh = B.make_shape(Tm, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                              B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32)
            m_shapes.append(sh)
            m_params.append(B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"][sl]))
            m_ys.append(y[sl])
            m_ws.append(B.alloc_workspace(sh, True))
            m_dys.append(dev["dy"][sl])
            fl = torch.zeros(total, dtype=torch.float32, device="cuda")
            gm = {n: fl[off:off + size] for n, (off, size) in offsets.items()}
            if want_dx:
                gm["d_x"] = g["d_x"][sl]
            m_keep.append((fl, gm))
            m_grads.append(B.make_grads(accumulate=0, **gm))

        def step():                        # noqa: F811
            B.mixlora_multi_ffn_forward(m_shapes, m_params, m_ys, m_ws)
            for m in range(M):
                B.mixlora_aux_loss(m_shapes[m], m_ws[m], AUX_COEF, loss)
            B.mixlora_multi_ffn_backward(m_shapes, m_params, m_dys, [AUX_COEF] * M, m_ws, m_grads)
            if use_dist:
                for fl, _ in m_keep:
                    dist.all_reduce(fl)

    if args.layer and M == 1 and want_dx:
        # the block inside its layer (Eq. 5 / Eq. 6): RMS normalisation in front, residual stream behind
        wn = torch.ones(w.d_model, dtype=act, device="cuda")
        xn = torch.empty(w.tokens, w.d_model, dtype=act, device="cuda")
        inv_rms = torch.empty(w.tokens, dtype=torch.float32, device="cuda")

        def step():                        # noqa: F811
            B.mixlora_layer_forward(shape, params, wn, 1e-5, xn, inv_rms, y, ws)
            B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
            B.mixlora_layer_backward(shape, params, wn, 1e-5, xn, inv_rms, dev["dy"], AUX_COEF, ws, grads)
            if use_dist:
                dist.all_reduce(flat)

    if args.forward_only:
        # the forward-only configuration: no backward pass, no gradient exchange
        def step():                        # noqa: F811
            B.mixlora_ffn_forward(shape, params, y, ws)
            B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        t1 = time.time()
        ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device="cuda")
        if use_dist:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item()), t0, t1

    B.mixlora_stage_timing(False)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    total_ms, t0, t1 = timed(step, args.steps, args.warmup)
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    launches = sum(v[1] for v in B.mixlora_stage_timing_read().values())
    launches_per_step = launches // (args.steps + args.warmup)
    status = B.mixlora_device_status(ws) if M == 1 else max(B.mixlora_device_status(x_) for x_ in m_ws)
    ms_per_step = total_ms / args.steps
    value = world * w.tokens / (ms_per_step * 1e-3)

    # per-stage device time over the same number of steps (events on the launching stream)
    B.mixlora_stage_timing(True)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize()
    stages = B.mixlora_stage_timing_read()
    B.mixlora_stage_timing(False)
    stage_ms = {n: v[0] / args.steps for n, v in stages.items()}

    # End to end through the same C-ABI calls with HOST buffers: every step's x and dy come from pinned host
    # memory and its y and loss go back to the host, all inside the timed region.  The copies of step i+1 run on
    # their own stream while step i computes (two device buffers per input), as a training loop would prefetch.
    hx = torch.from_numpy(tensors["x"]).to(act).pin_memory()
    hdy = torch.from_numpy(tensors["dy"]).to(act).pin_memory()
    hy = torch.empty(w.tokens, w.d_model, dtype=act).pin_memory()
    hloss = torch.empty(1, dtype=torch.float32).pin_memory()
    xb = [dev["x"], torch.empty_like(dev["x"])]
    dyb = [dev["dy"], torch.empty_like(dev["dy"])]
    yb = [y, torch.empty_like(y)]
    pb = [B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=xb[i]) for i in range(2)]
    h2d, d2h, main = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]

    def upload(bi):
        with torch.cuda.stream(h2d):
            h2d.wait_event(ev_done[bi])            # the step that last used this buffer has finished
            xb[bi].copy_(hx, non_blocking=True)
            dyb[bi].copy_(hdy, non_blocking=True)
            ev_in[bi].record(h2d)

    def run_e2e(steps):
        for bi in range(2):
            ev_done[bi].record(main)
        upload(0)
        for i in range(steps):
            bi = i & 1
            main.wait_event(ev_in[bi])
            if i + 1 < steps:
                upload(bi ^ 1)
            B.mixlora_ffn_forward(shape, pb[bi], yb[bi], ws)
            B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
            if not args.forward_only:
                B.mixlora_ffn_backward(shape, pb[bi], dyb[bi], AUX_COEF, ws, grads)
                if use_dist:
                    dist.all_reduce(flat)
            ev_done[bi].record(main)
            with torch.cuda.stream(d2h):
                d2h.wait_event(ev_done[bi])
                hy.copy_(yb[bi], non_blocking=True)
                hloss.copy_(loss, non_blocking=True)
        main.wait_stream(d2h)
        main.wait_stream(h2d)

    run_e2e(max(3, args.warmup))
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run_e2e(args.steps)
    e1.record()
    barrier()
    e2e_t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device="cuda")
    if use_dist:
        dist.all_reduce(e2e_t, op=dist.ReduceOp.MAX)
    e2e_ms = float(e2e_t.item())
    e2e_value = world * w.tokens / (e2e_ms / args.steps * 1e-3)
    h2d_bytes = hx.numel() * hx.element_size() + hdy.numel() * hdy.element_size()
    d2h_bytes = hy.numel() * hy.element_size() + 4

    if rank != 0:
        if use_dist:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    fl = stage_flops(w, want_dx)
    gemm_names = [n for n in fl if fl[n] > 0 and stage_ms.get(n, 0.0) > 0]
    dom = max(gemm_names, key=lambda n: stage_ms.get(n, 0.0))
    gemm_ms = sum(stage_ms.get(n, 0.0) for n in gemm_names)
    gemm_fl = sum(fl[n] for n in gemm_names)
    peak_tf = peaks["bf16_tflops_sustained"]       # the kernel is timed inside a long step
    dom_tf = fl[dom] / (stage_ms[dom] * 1e-3) / 1e12 if stage_ms.get(dom) else 0.0
    roofline = {"bound": "tensor", "kernel": dom, "achieved": dom_tf, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": dom_tf / peak_tf, "peak_source": peaks["source"] + " (sustained bf16)",
                "flops_per_launch": fl[dom], "ms_per_launch": stage_ms.get(dom), "traffic": None,
                "gemm_phases": {"tflops": gemm_fl / (gemm_ms * 1e-3) / 1e12 if gemm_ms else 0.0,
                                "frac": (gemm_fl / (gemm_ms * 1e-3) / 1e12 / peak_tf) if gemm_ms else 0.0,
                                "ms": gemm_ms, "share_of_step": gemm_ms / sum(stage_ms.values())}}

    # HBM-bound stages: algorithmic bytes / stage time against the measured copy bandwidth
    T_, d_, f_, k_, N_, r_ = w.tokens, w.d_model, w.d_ff, w.top_k, w.n_experts, w.rank
    E = 2 if bf16 else 4
    hbm_bytes = {
        "router": T_ * d_ * E + N_ * d_ * 4 + T_ * N_ * 4 * 2,
        "lora_b_swiglu": (T_ * f_ * 2 + T_ * k_ * f_) * E,                      # G, U once per token + h per slot
        "combine_h": (T_ * k_ * f_ + T_ * f_) * E,
        "swiglu_bwd": (T_ * f_ * 3 + T_ * k_ * f_ * 2) * E,                     # G, U, D once + da, db per slot
        "combine_bwd": (2 * T_ * k_ * f_ + 2 * T_ * f_) * E if want_dx else 0,
    }
    hbm = {n: {"gbs": round(bts / (stage_ms[n] * 1e-3) / 1e9, 1), "frac": round(bts / (stage_ms[n] * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
               "algorithmic_mb": round(bts / 1e6, 1)}
           for n, bts in hbm_bytes.items() if bts and stage_ms.get(n)}
    roofline["hbm_stages"] = hbm
    roofline["hbm_peak_gbs"] = peaks["hbm_gbs"]
    # DRAM bytes (read + write) of the frozen-projection launches, from one single-pass ncu capture of this command's
    # workload at full size (summary under profiles/); other workloads have no capture
    measured_dram = {"gemm_gate_up": 905.3e6, "gemm_down": 905.9e6, "gemm_dgrad_down": 463.9e6, "gemm_dx": 2110.0e6}
    algorithmic_dram = {"gemm_gate_up": (T_ * d_ + 2 * f_ * d_ + 2 * T_ * f_) * E,
                        "gemm_down": (T_ * f_ + f_ * d_ + T_ * d_) * E,
                        "gemm_dgrad_down": (T_ * d_ + f_ * d_ + T_ * f_) * E,
                        "gemm_dx": (2 * T_ * f_ + 2 * f_ * d_ + T_ * d_) * E}
    if w.name == synth.c3().name and want_dx and M == 1 and not args.layer and bf16 and not args.forward_only:
        roofline["traffic"] = measured_dram[dom]
        roofline["traffic_note"] = ("dram__bytes_read.sum + dram__bytes_write.sum of the %s launch at this size; its "
                                    "operands and result are %.1f MB" % (dom, algorithmic_dram[dom] / 1e6))
    else:
        roofline["traffic_note"] = "null: the DRAM counters were taken on the default workload only"

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sample = args.cpu_sample
        sec = oracle_sample(w, tensors, sample, want_dx)
        cpu_baseline = {"value": sample / sec, "unit": UNIT, "cores": threads_used(), "kind": "oracle",
                        "sample": f"one oracle pass (forward + aux + backward) over the first {sample} tokens of the "
                                  f"workload at full d_model/d_ff, {sec:.1f} s"}

    line = {
        "metric": METRIC if not args.forward_only else "mixlora_ffn_fwd_tokens_per_s", "value": value, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "tokens_per_gpu": w.tokens, "d_model": w.d_model, "d_ff": w.d_ff,
                   "n_experts": w.n_experts, "top_k": w.top_k, "rank": w.rank, "lora_alpha": w.lora_alpha,
                   "backward_dx": want_dx, "aux_coef": AUX_COEF, "adapters": M, "layer_slice": bool(args.layer and M == 1 and want_dx),
                   "parallelism": f"dp{world} over tokens" + (", NCCL all-reduce of LoRA/router grads beside the dx product" if use_dist else ""),
                   "l2": "inputs larger than L2 (weights 270 MB + activations > 126 MB), no flush"},
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes,
                "ms_per_step": e2e_ms / args.steps,
                "note": "x, dy from pinned host memory and y, loss back to it every step; copies of step i+1 overlap step i"},
        "gpu_launches": launches_per_step * args.steps, "gpu_launches_per_step": launches_per_step,
        "stage_ms": {n: round(v, 4) for n, v in stage_ms.items()}, "device_status": status, "clocks": clocks,
    }
    print(json.dumps(line))
    if use_dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--no-dx", action="store_true")
    ap.add_argument("--forward-only", action="store_true",
                    help="time the forward pass and the aux loss only (the forward-only configuration); the metric is "
                         "then named mixlora_ffn_fwd_tokens_per_s")
    ap.add_argument("--force-dist", action="store_true",
                    help="with one rank, still go through the NCCL gradient all-reduce path (plumbing check)")
    ap.add_argument("--layer", action="store_true",
                    help="time the block inside its layer (RMSNorm in front, residual behind) instead of the block alone")
    ap.add_argument("--models", type=int, default=1,
                    help="split the batch over this many adapters sharing the frozen FFN (multi-model calls); the "
                         "end-to-end leg still runs the single-model calls")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample", type=int, default=4096, help="tokens of the oracle's timed sample")
    ap.add_argument("--ref-sample", type=int, default=0,
                    help="tokens per step of --impl reference (0 = sized so that the run takes about two minutes)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
