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

DRAM_CAPTURE = "profiles/c3_step_dram_bytes.md"
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


def config_of(w: synth.Workload, args, world: int, use_dist: bool) -> dict:
    """The `config` object of the JSON line; both arms (the CUDA library and the CPU oracle) print the same keys."""
    want_dx = not args.no_dx
    M = max(1, args.models)
    return {"workload": w.name, "tokens_per_gpu": w.tokens, "d_model": w.d_model, "d_ff": w.d_ff,
            "n_experts": w.n_experts, "top_k": w.top_k, "rank": w.rank, "lora_alpha": w.lora_alpha,
            "backward_dx": want_dx, "aux_coef": AUX_COEF, "adapters": M,
            "layer_slice": bool(args.layer and M == 1 and want_dx),
            "variant": "mixdora" if getattr(args, "dora", False) else "mixlora",
            "parallelism": f"dp{world} over tokens" + (", aux statistics (2N floats) and LoRA/router gradients "
                                                        "all-reduced over NCCL, the latter beside the dx product"
                                                        if use_dist else ""),
            "l2": "inputs larger than L2 (weights 270 MB + activations > 126 MB), no flush; a flushed variant is "
                  "reported in step_ms_l2_flushed"}


# ----------------------------------------------------------------------------------------
# flop / byte model of the stages (per step)
# ----------------------------------------------------------------------------------------
def stage_flops(w: synth.Workload, want_dx: bool, executed: bool = False) -> dict:
    """Flops of the four frozen-projection launches.  Algorithmic: what the step needs, a slot's low-rank terms
    counted for its own expert only (k r columns per token).  Executed: what the launches compute, with the low-rank
    columns of every expert riding along (N r per token)."""
    T, d, f, N, k, r = w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank
    U = 2.0 * T * d * f
    cols = (N if executed else k) * r
    NR = ((N + 7) // 8 * 8) if executed else N
    fl = {
        "gemm_gate_up": 2 * U + 2 * 2.0 * T * d * cols,        # W1, W3 once per token + LoRA-A
        "gemm_down": U + 2.0 * T * cols * d,                   # W2 on the gate-weighted sum + LoRA-B down
        "gemm_dgrad_down": U + 2.0 * T * d * cols,             # dy W2 + B_d^T dy
        "gemm_dx": (2 * U + 2 * 2.0 * T * cols * d + 2.0 * T * NR * d) if want_dx else 0.0,
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
        "config": config_of(w, args, 1, False),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} tokens of the workload per step, full d_model/d_ff, forward + aux + "
                                   f"backward with dx, float64 numpy",
                         "role": "this run (the reference arm: a bounded sample per step so that any --steps ends in "
                                 "minutes); the stated CPU baseline is the cpu_baseline of the CUDA arm's line, one "
                                 "oracle pass over 4096 tokens"},
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
    if world != max(1, args.gpus) and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); reporting n_gpus = {world}",
              file=sys.stderr)
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

    def compute(params_, y_, dy_):
        B.mixlora_ffn_forward(shape, params_, y_, ws)
        B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
        B.mixlora_ffn_backward(shape, params_, dy_, AUX_COEF, ws, grads)

    if use_dist:
        # data-parallel sum of the LoRA and router gradients (one flat buffer, one NCCL all-reduce) on a second
        # stream: it starts when the parameter gradients are enqueued and runs beside the input-gradient product
        comm = torch.cuda.Stream()
        ev_ready = torch.cuda.Event()
        ev_ready.record()

        aux_sums = torch.zeros(2 * w.n_experts, dtype=torch.float32, device="cuda")   # probability sums, counts

        def compute(params_, y_, dy_):     # noqa: F811
            B.mixlora_ffn_forward(shape, params_, y_, ws)
            # Eq. 8-9 are fractions of the whole batch: the shards' sums are added (2N floats) before the loss
            B.mixlora_aux_stats(shape, ws, aux_sums[:w.n_experts], aux_sums[w.n_experts:])
            dist.all_reduce(aux_sums)
            B.mixlora_aux_loss_global(shape, ws, AUX_COEF, aux_sums[:w.n_experts], aux_sums[w.n_experts:],
                                      world * w.tokens, loss)
            B.mixlora_ffn_backward_overlap(shape, params_, dy_, AUX_COEF, ws, grads, ev_ready)
            comm.wait_event(ev_ready)
            with torch.cuda.stream(comm):
                dist.all_reduce(flat)
            torch.cuda.current_stream().wait_stream(comm)

    def step():
        compute(params, y, dev["dy"])

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

    if args.dora:
        # MixDoRA (Section 4.1 / Table 1): the same step with every expert's LoRA replaced by DoRA.  Magnitudes start,
        # as DoRA's do, from the row norms of the frozen weights, here times a factor in [0.8, 1.2].
        gen = torch.Generator(device="cuda").manual_seed(w.seed + 7)

        def mag(wt):
            base = wt.float().norm(dim=1)
            return (base[None, :] * (0.8 + 0.4 * torch.rand(w.n_experts, base.numel(), generator=gen, device="cuda"))
                    ).contiguous()

        m_dev = [mag(dev["w_gate"]), mag(dev["w_up"]), mag(dev["w_down"])]
        dm_dev = [torch.zeros_like(v) for v in m_dev]
        magn, dmagn = B.make_dora(*m_dev), B.make_dora_grads(*dm_dev)
        ws = B.alloc_dora_workspace(shape, True)

        def compute(params_, y_, dy_):     # noqa: F811
            B.mixlora_dora_ffn_forward(shape, params_, magn, y_, ws)
            B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
            B.mixlora_dora_ffn_backward(shape, params_, magn, dy_, AUX_COEF, ws, grads, dmagn)

        def step():                        # noqa: F811
            compute(params, y, dev["dy"])

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

    # every step with its own pair of events: median and minimum beside the mean of the headline loop; then the same
    # with L2 flushed before each step (a buffer larger than L2 is overwritten outside the timed pair)
    def per_step_times(flush):
        scratch = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if flush else None
        evs = []
        for _ in range(args.steps):
            if flush:
                scratch.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step()
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        ts = sorted(a.elapsed_time(b) for a, b in evs)
        return {"median": round(ts[len(ts) // 2], 4), "min": round(ts[0], 4), "mean": round(sum(ts) / len(ts), 4)}

    step_ms = per_step_times(False)
    step_ms_flushed = per_step_times(True)

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
            if args.forward_only:
                B.mixlora_ffn_forward(shape, pb[bi], yb[bi], ws)
                B.mixlora_aux_loss(shape, ws, AUX_COEF, loss)
            else:
                compute(pb[bi], yb[bi], dyb[bi])
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
    fl_exec = stage_flops(w, want_dx, executed=True)
    gemm_names = [n for n in fl if fl[n] > 0 and stage_ms.get(n, 0.0) > 0]
    dom = max(gemm_names, key=lambda n: stage_ms.get(n, 0.0))
    gemm_ms = sum(stage_ms.get(n, 0.0) for n in gemm_names)
    gemm_fl = sum(fl[n] for n in gemm_names)
    # The peak that applies depends on how long the GPU has been under load: a timed region well under a second
    # runs at the boost clock (the burst figure), a seconds-long one under the power cap (the sustained figure).
    # The stage timing above runs right after the headline loop and is as long, so it is judged the same way.
    burst = total_ms < 1000.0
    peak_tf = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    dom_tf = fl[dom] / (stage_ms[dom] * 1e-3) / 1e12 if stage_ms.get(dom) else 0.0
    gemm_tf = gemm_fl / (gemm_ms * 1e-3) / 1e12 if gemm_ms else 0.0
    roofline = {"bound": "tensor", "kernel": dom, "achieved": dom_tf, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": dom_tf / peak_tf,
                "peak_source": "%s (%s bf16: the timed region is %.2f s)" % (peaks["source"], "burst" if burst else "sustained",
                                                                             total_ms * 1e-3),
                "frac_of_burst": dom_tf / peaks["bf16_tflops"], "frac_of_sustained": dom_tf / peaks["bf16_tflops_sustained"],
                "sm_mhz_median": clocks.get("sm_mhz") if clocks else None,
                "flops_per_launch": fl[dom], "flops_executed_per_launch": fl_exec[dom],
                "ms_per_launch": stage_ms.get(dom), "traffic": None,
                "gemm_phases": {"tflops": gemm_tf, "frac": gemm_tf / peak_tf,
                                "frac_of_burst": gemm_tf / peaks["bf16_tflops"],
                                "frac_of_sustained": gemm_tf / peaks["bf16_tflops_sustained"],
                                "ms": gemm_ms, "share_of_step": gemm_ms / sum(stage_ms.values())}}
    roofline["check"] = "ok" if roofline["frac"] <= 1.02 else "frac above 1.02: the peak and the timed region do not match"

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
    measured_dram = {"gemm_gate_up": 876.4e6, "gemm_down": 901.8e6, "gemm_dgrad_down": 462.8e6, "gemm_dx": 1767.2e6}
    algorithmic_dram = {"gemm_gate_up": (T_ * d_ + 2 * f_ * d_ + 2 * T_ * f_) * E,
                        "gemm_down": (T_ * f_ + f_ * d_ + T_ * d_) * E,
                        "gemm_dgrad_down": (T_ * d_ + f_ * d_ + T_ * f_) * E,
                        "gemm_dx": (2 * T_ * f_ + 2 * f_ * d_ + T_ * d_) * E}
    if (w.name == synth.c3().name and want_dx and M == 1 and not args.layer and bf16 and not args.forward_only
            and not args.dora):
        roofline["traffic"] = measured_dram[dom]
        roofline["traffic_note"] = ("constant from %s (one single-pass ncu capture of this command's workload, not "
                                    "measured in this run): dram__bytes_read.sum + dram__bytes_write.sum of the %s "
                                    "launch; its operands and result are %.1f MB"
                                    % (DRAM_CAPTURE, dom, algorithmic_dram[dom] / 1e6))
    else:
        roofline["traffic_note"] = "null: the DRAM counters were taken on the default workload only"

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sample = args.cpu_sample
        sec = oracle_sample(w, tensors, sample, want_dx)
        cpu_baseline = {"value": sample / sec, "unit": UNIT, "cores": threads_used(), "kind": "oracle",
                        "sample": f"one oracle pass (forward + aux + backward) over the first {sample} tokens of the "
                                  f"workload at full d_model/d_ff, {sec:.1f} s",
                        "role": "the stated CPU baseline (the line of --impl reference times the same oracle on a "
                                "smaller per-step sample)"}

    line = {
        "metric": METRIC if not args.forward_only else "mixlora_ffn_fwd_tokens_per_s", "value": value, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
        "config": config_of(w, args, world, use_dist),
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes,
                "ms_per_step": e2e_ms / args.steps,
                "note": "x, dy from pinned host memory and y, loss back to it every step; copies of step i+1 overlap step i"},
        "gpu_launches": launches_per_step * args.steps, "gpu_launches_per_step": launches_per_step,
        "stage_ms": {n: round(v, 4) for n, v in stage_ms.items()}, "step_ms": step_ms,
        "step_ms_l2_flushed": step_ms_flushed, "device_status": status, "clocks": clocks,
    }
    print(json.dumps(line))
    if use_dist:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------
# --gpus N without a launcher: start the ranks here
# ----------------------------------------------------------------------------------------
def spawn_ranks(args) -> int:
    """Re-runs this script as `args.gpus` ranks under torch.distributed.run (one process per GPU, rendezvous on
    127.0.0.1) and returns the launcher's exit code.  Rank 0 prints the JSON line."""
    if not args.stub:
        import torch
        seen = torch.cuda.device_count()
        if args.gpus > seen:
            raise SystemExit(f"--gpus {args.gpus}, but {seen} CUDA device(s) are visible")
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's rank count can be read from its log (stderr)
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("OMP_NUM_THREADS", "4")
    return subprocess.call(cmd, env=env)


def run_stub(args):
    """Host-only check of the multi-rank plumbing (no GPU, gloo): the same rendezvous, barriers, max-over-ranks
    timing and rank-0 JSON line as the CUDA leg around a stand-in step that only does the step's two exchanges
    (2N floats of auxiliary statistics, the flat gradient buffer).  It measures nothing."""
    import torch
    import torch.distributed as dist
    from paper_2404_15159_b200 import dp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    w = workload_by_name(args.workload)
    offsets, total = dp.flat_grad_layout(64, 96, w.n_experts, 8)
    flat = torch.full((total,), float(rank + 1), dtype=torch.float32)
    aux = torch.full((2 * w.n_experts,), 1.0, dtype=torch.float32)

    def step():
        time.sleep(0.001)
        if world > 1:
            dist.all_reduce(aux)
            dist.all_reduce(flat)

    for _ in range(args.warmup):
        step()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    if world > 1:
        dist.barrier()
    ms = torch.tensor([(time.perf_counter() - t0) * 1e3], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    if rank == 0:
        per = float(ms.item()) / args.steps
        print(json.dumps({"impl": "stub", "metric": METRIC, "value": world * w.tokens / (per * 1e-3), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "none",
                          "data": "none", "config": config_of(w, args, world, world > 1), "gpu_launches": 0,
                          "note": "plumbing check on CPU ranks; not a measurement"}))
    if world > 1:
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
    ap.add_argument("--dora", action="store_true",
                    help="time the MixDoRA variant of the step (mixlora_dora_ffn_forward / _backward)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample", type=int, default=4096, help="tokens of the oracle's timed sample")
    ap.add_argument("--ref-sample", type=int, default=0,
                    help="tokens per step of --impl reference (0 = sized so that the run takes about two minutes)")
    ap.add_argument("--stub", action="store_true",
                    help="host-only check of the multi-rank plumbing: gloo ranks on CPU around a stand-in step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: become the launcher (one rank per GPU), the ranks print the line
        raise SystemExit(spawn_ranks(args))
    if args.stub:
        run_stub(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
