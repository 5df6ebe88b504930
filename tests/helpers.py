"""Shared helpers of the GPU parity tests: run the CUDA library through its C ABI and the
CPU oracle on the same seeded tensors, and compare."""
from __future__ import annotations

import numpy as np

from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

# Routing is compared bit for bit on every token whose deciding logit gap (float64, the oracle's) is at least
# 1e-4, the threshold at which the library itself flags a token; the 10 % on top covers the fp32 rounding of the
# library's logits (a few 1e-6 on logits of order one), as the flag check in check_parity does.
ROUTE_MARGIN = 1.1e-4

GRAD_NAMES = ("d_a_gate", "d_b_gate", "d_a_up", "d_b_up", "d_a_down", "d_b_down", "d_w_router", "d_router_bias")
ACT_NAMES = ("x", "dy", "w_gate", "w_up", "w_down", "a_gate", "b_gate", "a_up", "b_up", "a_down", "b_down")


def rel_err(got, ref) -> float:
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    denom = np.abs(ref).max()
    if denom == 0:
        return float(np.abs(got).max())
    return float(np.abs(got - ref).max() / denom)


def gpu_run(w: synth.Workload, tensors: dict, backward=True, want_dx=True, aux_coef=0.01, renormalize=1,
            aux_f_mode=0, accumulate=0, grads_init=None, repeats=1, overlap=False):
    """Forward (+ aux loss, + backward) on the GPU through the C ABI.  Returns numpy arrays."""
    import torch
    from paper_2404_15159_b200 import binding as B

    bf16 = w.dtype == "bf16"
    act = torch.bfloat16 if bf16 else torch.float32
    dev = {}
    for n, v in tensors.items():
        if v is None:
            dev[n] = None
        elif np.size(v) == 0:
            dev[n] = torch.empty(8, dtype=act if n in ACT_NAMES else torch.float32, device="cuda")
        elif n in ACT_NAMES:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v)).to("cuda").to(act).contiguous()
        else:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v, np.float32)).to("cuda")
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                         B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32, renormalize, aux_f_mode)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, backward)
    y = torch.empty(max(w.tokens, 1), w.d_model, dtype=act, device="cuda")[: w.tokens]
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    F = torch.zeros(w.n_experts, dtype=torch.float32, device="cuda")
    P = torch.zeros(w.n_experts, dtype=torch.float32, device="cuda")
    out = {}
    g = {}
    for _ in range(repeats):
        B.mixlora_ffn_forward(shape, params, y if w.tokens else torch.empty(8, dtype=act, device="cuda"), ws)
        B.mixlora_aux_loss(shape, ws, aux_coef, loss, F, P)
        if backward:
            g = {}
            for n in GRAD_NAMES:
                ref = tensors[n[2:]] if n != "d_router_bias" else np.zeros(w.n_experts, np.float32)
                if grads_init is not None:
                    g[n] = torch.from_numpy(np.ascontiguousarray(grads_init[n], np.float32)).to("cuda")
                else:
                    g[n] = torch.full(tuple(np.shape(ref)), float("nan"), dtype=torch.float32, device="cuda")
            if want_dx:
                g["d_x"] = torch.full((max(w.tokens, 1), w.d_model), float("nan"), dtype=act, device="cuda")[: w.tokens]
            grads = B.make_grads(accumulate=accumulate, **{n: (v if v.numel() else torch.empty(8, device="cuda"))
                                                           for n, v in g.items()})
            dy_dev = dev["dy"] if w.tokens else torch.empty(8, dtype=act, device="cuda")
            if overlap:
                # the variant that signals when the parameter gradients are enqueued: a second stream copies them
                # at that point, while the input-gradient product is still to run
                ev = torch.cuda.Event()
                ev.record()
                side = torch.cuda.Stream()
                B.mixlora_ffn_backward_overlap(shape, params, dy_dev, aux_coef, ws, grads, ev)
                side.wait_event(ev)
                with torch.cuda.stream(side):
                    snap = {n: v.clone() for n, v in g.items() if n != "d_x"}
                torch.cuda.current_stream().wait_stream(side)
                for n, v in snap.items():
                    out["snap_" + n] = v
            else:
                B.mixlora_ffn_backward(shape, params, dy_dev, aux_coef, ws, grads)
    torch.cuda.synchronize()
    out["status"] = B.mixlora_device_status(ws)
    out["y"] = y.float().cpu().numpy()
    out["loss"] = float(loss.item())
    out["F"] = F.cpu().numpy()
    out["P"] = P.cpu().numpy()
    view = B.mixlora_routing_view(shape, ws)
    for n, v in view.items():
        out[n] = v.cpu().numpy().copy()
    for n, v in g.items():
        out[n] = v.float().cpu().numpy()
    for n in [n for n in out if n.startswith("snap_")]:
        out[n] = out[n].float().cpu().numpy()
    return out


def oracle_run(w: synth.Workload, tensors: dict, gpu_out: dict | None, backward=True, want_dx=True, aux_coef=0.01,
               renormalize=True, aux_f_mode=0):
    """Oracle on the same tensors.  Where the GPU flagged a low routing margin and chose
    differently, the oracle is re-run with the GPU's choice forced for those tokens only."""
    params = synth.params_of(tensors)
    y, saved = orc.ffn_forward(tensors["x"], params, w.top_k, w.lora_alpha, renormalize=renormalize)
    info = dict(forced=0, flagged=0)
    if gpu_out is not None and w.tokens > 0:
        idx = saved["route"]["expert_idx"]
        low = saved["route"]["margin"] < ROUTE_MARGIN
        info["flagged"] = int(low.sum())
        diff = (gpu_out["expert_idx"] != idx).any(axis=1)
        assert not (diff & ~low).any(), "expert choice differs on a token with a clear margin"
        if diff.any():
            assert_near_tie(saved["route"]["logits"], idx, gpu_out["expert_idx"], diff, ROUTE_MARGIN)
            forced = idx.copy()
            forced[diff] = gpu_out["expert_idx"][diff]
            info["forced"] = int(diff.sum())
            y, saved = orc.ffn_forward(tensors["x"], params, w.top_k, w.lora_alpha, renormalize=renormalize,
                                       forced_expert_idx=forced)
    res = dict(y=y, saved=saved, info=info)
    loss, F, P = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], aux_coef, aux_f_mode) \
        if w.tokens > 0 else (0.0, np.zeros(w.n_experts), np.zeros(w.n_experts))
    res.update(loss=loss, F=F, P=P)
    if backward:
        res["grads"] = orc.ffn_backward(tensors["x"], params, tensors["dy"], saved, aux_coef=aux_coef,
                                        aux_f_mode=aux_f_mode, want_dx=want_dx)
    return res


def assert_near_tie(logits, idx, other_idx, rows, slack):
    """Where another choice of experts is accepted for a token, it must be one the near-tie allows: distinct
    experts, the j-th of which has a logit within `slack` of the oracle's own j-th choice."""
    for t in np.flatnonzero(rows):
        chosen = other_idx[t]
        assert len(set(chosen.tolist())) == len(chosen) and chosen.min() >= 0 and chosen.max() < logits.shape[1]
        gap = np.abs(logits[t, chosen.astype(np.int64)] - logits[t, idx[t].astype(np.int64)]).max()
        assert gap <= slack, f"token {t}: accepted choice {chosen} is {gap:.3e} away from the oracle's {idx[t]}"


def check_parity(w, gpu, ref, tol, backward=True, want_dx=True, report=None):
    """Bit-exact routing (flagged tokens excepted, handled in oracle_run), tolerance on values."""
    route, disp = ref["saved"]["route"], ref["saved"]["disp"]
    assert gpu["status"] == 0
    np.testing.assert_array_equal(gpu["expert_idx"], route["expert_idx"])
    np.testing.assert_array_equal(gpu["perm"], disp["perm"])
    np.testing.assert_array_equal(gpu["seg_off"], disp["seg_off"])
    # every token the oracle sees with a small margin must carry the flag (threshold 1e-4, with slack
    # for the fp32 logits), and no token with a wide margin may
    m = route["margin"]
    assert (gpu["low_margin"][m < 0.9e-4] == 1).all()
    assert (gpu["low_margin"][m > 1.1e-4] == 0).all()
    errs = {}
    errs["probs"] = rel_err(gpu["probs"], route["probs"])
    errs["gates"] = rel_err(gpu["gates"], route["gates"])
    errs["y"] = rel_err(gpu["y"], ref["y"])
    errs["loss"] = abs(gpu["loss"] - ref["loss"]) / max(abs(ref["loss"]), 1e-30) if ref["loss"] else abs(gpu["loss"])
    errs["F"] = rel_err(gpu["F"], ref["F"])
    errs["P"] = rel_err(gpu["P"], ref["P"])
    if backward:
        for n in GRAD_NAMES:
            errs[n] = rel_err(gpu[n], ref["grads"][n])
        if want_dx:
            errs["d_x"] = rel_err(gpu["d_x"], ref["grads"]["d_x"])
    if report is not None:
        report.update(errs)
    router_tol = 1e-5
    for n, e in errs.items():
        lim = router_tol if n in ("probs", "gates", "F", "P", "loss") else tol
        assert e <= lim, f"{w.name}: {n} relative error {e:.3e} > {lim:.1e}  (all: {errs})"
    return errs
