"""MixDoRA on the GPU (through the C ABI) against its CPU oracle on the same seeded tensors: routing bit-exact
on tokens with a clear margin, outputs and every gradient (LoRA matrices, magnitudes, router, x) within the
tolerances of the MixLoRA parity tests."""
import numpy as np
import pytest

import helpers
from oracle import mixdora_oracle as dora
from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu

MAG = ("gate", "up", "down")


def small(name, dtype="bf16", **kw):
    base = dict(tokens=300, d_model=256, d_ff=688, n_experts=8, top_k=2, rank=16, lora_alpha=32.0, dtype=dtype,
                std_frozen=0.05, std_a=0.06, std_b=0.05, seed=synth.BASE_SEED + 300)
    base.update(kw)
    return synth.Workload(name, **base)


def magnitudes(w, t, spread):
    """Magnitudes around the current row norms (DoRA starts from the norm of the frozen weight): norm * U(1 - spread,
    1 + spread), drawn from a generator of their own."""
    rng = np.random.default_rng(w.seed + 7)
    n = dora.all_norms(synth.params_of(t), w.lora_alpha)
    return {k: (n[k] * rng.uniform(1 - spread, 1 + spread, n[k].shape)).astype(np.float32) for k in MAG}


def gpu_dora(w, t, m, aux_coef, want_dx=True, accumulate=0, init=None):
    import torch
    from paper_2404_15159_b200 import binding as B

    bf16 = w.dtype == "bf16"
    act = torch.bfloat16 if bf16 else torch.float32
    dev = {}
    for n, v in t.items():
        if v is None:
            dev[n] = None
        elif np.size(v) == 0:                  # no tokens: any valid pointer will do
            dev[n] = torch.empty(8, dtype=act if n in helpers.ACT_NAMES else torch.float32, device="cuda")
        elif n in helpers.ACT_NAMES:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v)).cuda().to(act).contiguous()
        else:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v, np.float32)).cuda()
    md = {k: torch.from_numpy(m[k]).cuda() for k in MAG}
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                         B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32, 1, 0)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    magn = B.make_dora(md["gate"], md["up"], md["down"])
    ws = B.alloc_dora_workspace(shape, True)
    y = torch.empty(max(w.tokens, 1), w.d_model, dtype=act, device="cuda")[: w.tokens]
    B.mixlora_dora_ffn_forward(shape, params, magn, y if w.tokens else torch.empty(8, dtype=act, device="cuda"), ws)
    loss = torch.zeros(1, device="cuda")
    B.mixlora_aux_loss(shape, ws, aux_coef, loss)
    g = {}
    for n in helpers.GRAD_NAMES:
        ref = t[n[2:]] if n != "d_router_bias" else np.zeros(w.n_experts, np.float32)
        g[n] = torch.full(tuple(np.shape(ref)), float("nan") if not accumulate else init, device="cuda")
    gm = {k: torch.full(tuple(m[k].shape), float("nan") if not accumulate else init, device="cuda") for k in MAG}
    if want_dx:
        g["d_x"] = torch.full((max(w.tokens, 1), w.d_model), float("nan"), dtype=act, device="cuda")[: w.tokens]
    B.mixlora_dora_ffn_backward(shape, params, magn, dev["dy"], aux_coef, ws, B.make_grads(accumulate=accumulate, **g),
                                B.make_dora_grads(gm["gate"], gm["up"], gm["down"]))
    torch.cuda.synchronize()
    out = {n: v.float().cpu().numpy() for n, v in g.items()}
    out.update({"d_m_" + k: gm[k].cpu().numpy() for k in MAG})
    out["y"] = y.float().cpu().numpy()
    out["loss"] = float(loss.item())
    out["status"] = B.mixlora_device_status(ws)
    out.update({n: v.cpu().numpy().copy() for n, v in B.mixlora_routing_view(shape, ws).items()})
    return out


def check(w, tol, spread=0.3, aux_coef=0.01, want_dx=True):
    t = synth.generate(w)
    m = magnitudes(w, t, spread)
    gpu = gpu_dora(w, t, m, aux_coef, want_dx)
    assert gpu["status"] == 0
    p = synth.params_of(t)
    y, saved = dora.ffn_forward(t["x"], p, m, w.top_k, w.lora_alpha)
    route = saved["route"]
    diff = (gpu["expert_idx"] != route["expert_idx"]).any(axis=1)
    assert not (diff & (route["margin"] >= helpers.ROUTE_MARGIN)).any()
    if diff.any():
        helpers.assert_near_tie(route["logits"], route["expert_idx"], gpu["expert_idx"], diff, helpers.ROUTE_MARGIN)
        y, saved = dora.ffn_forward(t["x"], p, m, w.top_k, w.lora_alpha, forced_expert_idx=gpu["expert_idx"])
    np.testing.assert_array_equal(gpu["perm"], saved["disp"]["perm"])
    g = dora.ffn_backward(t["x"], p, m, t["dy"], saved, aux_coef=aux_coef, want_dx=want_dx)
    loss_ref, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], aux_coef, 0)
    errs = {"y": helpers.rel_err(gpu["y"], y)}
    for n in helpers.GRAD_NAMES + tuple("d_m_" + k for k in MAG) + (("d_x",) if want_dx else ()):
        errs[n] = helpers.rel_err(gpu[n], g[n])
    assert abs(gpu["loss"] - loss_ref) <= 1e-5 * max(abs(loss_ref), 1e-30)
    for n, e in errs.items():
        assert e <= tol, f"{w.name}: {n} relative error {e:.3e} > {tol:.1e} (all: {errs})"
    return errs


@pytest.mark.parametrize("T", [1, 129, 300])
def test_fp32_check_mode(T):
    check(small(f"dora-fp32-T{T}", "fp32", tokens=T, rank=8, n_experts=4), 1e-4)


# bf16: the scaled SwiGLU runs on the grouped tensor-core kernel (the fp32 tests above take the SIMT kernels)
@pytest.mark.parametrize("N,k,r", [(1, 1, 8), (8, 2, 16), (4, 4, 32), (16, 2, 64), (8, 2, 128)])
def test_bf16_grid(N, k, r):
    check(small(f"dora-bf16-N{N}-k{k}-r{r}", n_experts=N, top_k=k, rank=r, lora_alpha=2.0 * r, std_a=1.0 / r), 2e-2)


def test_bf16_several_tiles_per_expert_ragged_width_no_dx():
    check(small("dora-slice", tokens=1111, d_model=512, d_ff=1376, std_frozen=0.02, std_a=1.0 / 16, std_b=0.01), 2e-2,
          want_dx=False)


def test_magnitudes_equal_to_the_norms_reproduce_the_mixlora_path():
    w = small("dora-as-lora", "fp32", rank=8, n_experts=4)
    t = synth.generate(w)
    m = magnitudes(w, t, 0.0)
    gpu = gpu_dora(w, t, m, 0.01)
    ref = helpers.gpu_run(w, t, aux_coef=0.01)
    for n in ("y", "d_x") + helpers.GRAD_NAMES:
        assert helpers.rel_err(gpu[n], ref[n]) < 1e-4, n


def test_zero_tokens_and_accumulation():
    w = small("dora-empty", "fp32", tokens=0, rank=8, n_experts=4)
    t = synth.generate(w)
    m = {k: np.ones(s, np.float32) for k, s in (("gate", (4, w.d_ff)), ("up", (4, w.d_ff)), ("down", (4, w.d_model)))}
    gpu = gpu_dora(w, t, m, 0.01, want_dx=False)
    assert gpu["status"] == 0 and all(np.all(gpu["d_m_" + k] == 0) for k in MAG)
    w = small("dora-accum", "fp32", rank=8, n_experts=4)
    t = synth.generate(w)
    m = magnitudes(w, t, 0.3)
    a = gpu_dora(w, t, m, 0.01)
    b = gpu_dora(w, t, m, 0.01, accumulate=1, init=0.5)
    for n in helpers.GRAD_NAMES + tuple("d_m_" + k for k in MAG):
        np.testing.assert_allclose(b[n], a[n] + 0.5, rtol=1e-5, atol=1e-6)


def test_llama2_7b_shape_1024_tokens_every_output():
    # the 7B-shaped block (d = 4096, f = 11008, 8 experts, top-2, rank 16) on the tensor-core products
    errs = check(synth.c3().with_(name="dora-7b-1024", tokens=1024), 2e-2)
    print("MixDoRA 7B shape, 1024 tokens:", {k: f"{v:.2e}" for k, v in errs.items()})
