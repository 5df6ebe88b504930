"""The block inside its transformer layer (Eq. 5 / Eq. 6): RMS normalisation in front of the MixLoRA block, the
residual stream added behind it, forward and backward, through the C ABI against the CPU oracle."""
import numpy as np
import pytest

import helpers
from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu

EPS = 1e-5


def norm_weight(w: synth.Workload):
    rng = np.random.default_rng(w.seed + 77)
    v = 1.0 + 0.2 * rng.standard_normal(w.d_model)
    return synth.round_to_bf16(v) if w.dtype == "bf16" else v.astype(np.float32).astype(np.float64)


def act_round(w):
    return synth.round_to_bf16 if w.dtype == "bf16" else (lambda a: np.asarray(a, np.float32).astype(np.float64))


def gpu_layer(w, t, wn, aux_coef=0.01, want_dx=True):
    import torch
    from paper_2404_15159_b200 import binding as B

    bf16 = w.dtype == "bf16"
    act = torch.bfloat16 if bf16 else torch.float32
    dev = {}
    for n, v in t.items():
        if v is None:
            dev[n] = None
        elif n in helpers.ACT_NAMES:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v)).to("cuda").to(act).contiguous()
        else:
            dev[n] = torch.from_numpy(np.ascontiguousarray(v, np.float32)).to("cuda")
    wn_d = torch.from_numpy(wn).to("cuda").to(act)
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                         B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, True)
    xn = torch.full((w.tokens, w.d_model), float("nan"), dtype=act, device="cuda")
    inv = torch.full((w.tokens,), float("nan"), dtype=torch.float32, device="cuda")
    h = torch.full((w.tokens, w.d_model), float("nan"), dtype=act, device="cuda")
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    g = {}
    for n in helpers.GRAD_NAMES:
        shp = (w.n_experts,) if n == "d_router_bias" else tuple(np.shape(t[n[2:]]))
        g[n] = torch.full(shp, float("nan"), dtype=torch.float32, device="cuda")
    if want_dx:
        g["d_x"] = torch.full((w.tokens, w.d_model), float("nan"), dtype=act, device="cuda")
    grads = B.make_grads(accumulate=0, **g)
    out = {}
    for _ in range(2):                                   # two calls in a row give the same bits
        B.mixlora_layer_forward(shape, params, wn_d, EPS, xn, inv, h, ws)
        B.mixlora_aux_loss(shape, ws, aux_coef, loss)
        B.mixlora_layer_backward(shape, params, wn_d, EPS, xn, inv, dev["dy"], aux_coef, ws, grads)
        torch.cuda.synchronize()
        cur = dict(h=h.float().cpu().numpy(), xn=xn.float().cpu().numpy(), inv_rms=inv.cpu().numpy(),
                   loss=float(loss.item()), **{n: v.float().cpu().numpy() for n, v in g.items()})
        if out:
            for n in cur:
                np.testing.assert_array_equal(cur[n], out[n])
        out = cur
    out["status"] = B.mixlora_device_status(ws)
    for n, v in B.mixlora_routing_view(shape, ws).items():
        out[n] = v.cpu().numpy().copy()
    return out


def routing_slack(w, t, wn):
    """Per token, how far a deciding logit gap can move because the library rounds the normalised input to its
    storage type from an fp32 value and the oracle from a float64 one.
    bf16 storage: an element changes only if its exact value lies so close to the midpoint of two neighbouring bf16
    values that the fp32 evaluation (three products, a reciprocal square root of a 2-ulp-accurate sum: at most
    16 fp32 ulps = 2^-20 relative) can land on the other side; it then moves by one bf16 ulp, and a gap between two
    logits by at most (max_e W_r[e, c] - min_e W_r[e, c]) times that.  The slack of a token is the sum over its
    ambiguous elements (most tokens have none).  fp32 storage: every element may differ by two fp32 ulps."""
    xn, _ = orc.rmsnorm(t["x"], wn, EPS)
    wr = np.asarray(t["w_router"], np.float64)
    spread = wr.max(axis=0) - wr.min(axis=0)                       # [d]
    mag = np.abs(xn)
    expo = np.floor(np.log2(np.where(mag > 0, mag, 1.0)))
    if w.dtype == "bf16":
        ulp = 2.0 ** (expo - 7)
        frac = np.mod(mag / ulp, 1.0)                              # position between the two neighbours, in ulps
        ambiguous = np.abs(frac - 0.5) * ulp <= mag * 2.0 ** -20
        return (ambiguous * ulp * spread[None, :]).sum(axis=1)
    ulp = 2.0 ** (expo - 23)
    return 2.0 * (ulp * spread[None, :]).sum(axis=1)


def oracle_layer(w, t, wn, gpu, aux_coef=0.01):
    params = synth.params_of(t)
    kw = dict(top_k=w.top_k, lora_alpha=w.lora_alpha, xn_round=act_round(w))
    h, saved = orc.layer_forward(t["x"], params, wn, EPS, **kw)
    idx = saved["route"]["expert_idx"]
    # bit-exact routing on every token whose deciding gap is at least 1e-4 (+10 % for the fp32 logits) plus what the
    # storage rounding of the normalised input can move it by, token by token
    slack = helpers.ROUTE_MARGIN + routing_slack(w, t, wn)
    low = saved["route"]["margin"] < slack
    diff = (gpu["expert_idx"] != idx).any(axis=1)
    assert not (diff & ~low).any(), "expert choice differs on a token with a clear margin"
    print(f"{w.name}: {int((slack > helpers.ROUTE_MARGIN * 1.01).sum())} of {w.tokens} tokens have an element on a "
          f"rounding boundary; {int(low.sum())} tokens inside their slack, {int(diff.sum())} routed differently")
    if diff.any():
        helpers.assert_near_tie(saved["route"]["logits"], idx, gpu["expert_idx"], diff, float(slack[diff].max()))
        forced = idx.copy()
        forced[diff] = gpu["expert_idx"][diff]
        h, saved = orc.layer_forward(t["x"], params, wn, EPS, forced_expert_idx=forced, **kw)
    loss, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], aux_coef)
    grads = orc.layer_backward(t["x"], params, wn, t["dy"], saved, aux_coef=aux_coef)
    return dict(h=h, saved=saved, loss=loss, grads=grads, forced=int(diff.sum()))


def compare(w, gpu, ref, tol):
    assert gpu["status"] == 0
    np.testing.assert_array_equal(gpu["expert_idx"], ref["saved"]["route"]["expert_idx"])
    np.testing.assert_array_equal(gpu["perm"], ref["saved"]["disp"]["perm"])
    errs = dict(inv_rms=helpers.rel_err(gpu["inv_rms"], ref["saved"]["inv_rms"]),
                xn=helpers.rel_err(gpu["xn"], ref["saved"]["xn"]),
                h=helpers.rel_err(gpu["h"], ref["h"]),
                loss=abs(gpu["loss"] - ref["loss"]) / abs(ref["loss"]))
    for n in helpers.GRAD_NAMES + ("d_x",):
        errs[n] = helpers.rel_err(gpu[n], ref["grads"][n])
    for n, e in errs.items():
        lim = 1e-5 if n == "inv_rms" else (1e-4 if n == "loss" else tol)
        assert e <= lim, f"{w.name}: {n} relative error {e:.3e} > {lim:.1e} (all: {errs})"
    return errs


def test_layer_fp32_check_mode_tiny_config():
    w = synth.c1()
    t = synth.generate(w)
    t["x"] = (t["x"] * 1.5 + 0.1).astype(np.float32).astype(np.float64)   # a residual stream is not unit-variance
    wn = norm_weight(w)
    gpu = gpu_layer(w, t, wn)
    compare(w, gpu, oracle_layer(w, t, wn, gpu), 1e-4)


@pytest.mark.parametrize("T,N,k,r", [(1000, 8, 2, 16), (257, 4, 1, 8), (640, 16, 2, 64)])
def test_layer_bf16(T, N, k, r):
    w = synth.Workload(f"layer-bf16-T{T}-N{N}-k{k}-r{r}", tokens=T, d_model=512, d_ff=1408, n_experts=N, top_k=k,
                       rank=r, lora_alpha=2.0 * r, dtype="bf16", seed=synth.BASE_SEED + 500 + T, std_frozen=0.03,
                       std_a=0.06, std_b=0.03)
    t = synth.generate(w)
    t["x"] = synth.round_to_bf16(t["x"] * 2.0)
    wn = norm_weight(w)
    gpu = gpu_layer(w, t, wn)
    compare(w, gpu, oracle_layer(w, t, wn, gpu), 2e-2)


def test_layer_with_a_dead_block_is_the_identity_on_the_residual_stream():
    # W_d = 0 and B_d = 0: h = z exactly, and dL/dz = dh exactly (the rounding of a sum with an exact zero)
    w = synth.Workload("layer-identity", tokens=300, d_model=256, d_ff=512, n_experts=4, top_k=2, rank=8,
                       lora_alpha=16.0, dtype="bf16", seed=synth.BASE_SEED + 600, std_frozen=0.03, std_a=0.06, std_b=0.03)
    t = synth.generate(w)
    t["w_down"] = np.zeros_like(t["w_down"])
    t["b_down"] = np.zeros_like(t["b_down"])
    wn = norm_weight(w)
    gpu = gpu_layer(w, t, wn, aux_coef=0.0)
    np.testing.assert_array_equal(gpu["h"], t["x"])
    np.testing.assert_array_equal(gpu["d_x"], t["dy"])


def test_layer_rejects_aliased_buffers_and_wide_models():
    import torch
    from paper_2404_15159_b200 import binding as B

    w = synth.Workload("layer-args", tokens=64, d_model=256, d_ff=512, n_experts=4, top_k=2, rank=8, lora_alpha=16.0,
                       dtype="bf16", seed=synth.BASE_SEED + 601, std_frozen=0.03, std_a=0.06, std_b=0.03)
    t = synth.generate(w)
    dev = {n: (torch.from_numpy(np.ascontiguousarray(v)).cuda().to(torch.bfloat16) if n in helpers.ACT_NAMES
               else torch.from_numpy(np.ascontiguousarray(v, np.float32)).cuda())
           for n, v in t.items() if v is not None}
    dev["router_bias"] = None
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, True)
    wn = torch.ones(w.d_model, dtype=torch.bfloat16, device="cuda")
    inv = torch.zeros(w.tokens, dtype=torch.float32, device="cuda")
    h = torch.zeros_like(dev["x"])
    with pytest.raises(B.MixLoraError) as e:
        B.mixlora_layer_forward(shape, params, wn, EPS, dev["x"], inv, h, ws)        # xn aliases z
    assert e.value.status == 1          # MIXLORA_ERR_INVALID_ARG
    wide = B.make_shape(8, 16384, 512, 4, 2, 8, 16.0)
    with pytest.raises(B.MixLoraError) as e:
        B.mixlora_layer_forward(wide, params, wn, EPS, h, inv, torch.zeros_like(h), ws)
    assert e.value.status == 2          # MIXLORA_ERR_UNSUPPORTED: wider than the norm kernels take


def test_layer_with_no_tokens_returns_zero_gradients():
    import torch
    from paper_2404_15159_b200 import binding as B

    w = synth.Workload("layer-empty", tokens=0, d_model=256, d_ff=512, n_experts=4, top_k=2, rank=8, lora_alpha=16.0,
                       dtype="bf16", seed=synth.BASE_SEED + 602, std_frozen=0.03, std_a=0.06, std_b=0.03)
    t = synth.generate(w.with_(tokens=8))
    act = torch.bfloat16
    dev = {n: (torch.from_numpy(np.ascontiguousarray(v)).cuda().to(act) if n in helpers.ACT_NAMES
               else torch.from_numpy(np.ascontiguousarray(v, np.float32)).cuda())
           for n, v in t.items() if v is not None}
    dev["router_bias"] = None
    shape = B.make_shape(0, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, True)
    wn = torch.ones(w.d_model, dtype=act, device="cuda")
    xn = torch.zeros(8, w.d_model, dtype=act, device="cuda")
    inv = torch.zeros(8, dtype=torch.float32, device="cuda")
    h = torch.zeros(8, w.d_model, dtype=act, device="cuda")
    g = {}
    for n in helpers.GRAD_NAMES:
        shp = (w.n_experts,) if n == "d_router_bias" else tuple(np.shape(t[n[2:]]))
        g[n] = torch.full(shp, float("nan"), dtype=torch.float32, device="cuda")
    g["d_x"] = torch.zeros(8, w.d_model, dtype=act, device="cuda")
    B.mixlora_layer_forward(shape, params, wn, EPS, xn, inv, h, ws)
    B.mixlora_layer_backward(shape, params, wn, EPS, xn, inv, dev["dy"], 0.01, ws, B.make_grads(accumulate=0, **g))
    torch.cuda.synchronize()
    assert B.mixlora_device_status(ws) == 0
    for n in helpers.GRAD_NAMES:
        assert not g[n].cpu().numpy().any(), n


def test_layer_full_size_sampled_tokens():
    # the 7B-shaped training configuration through the layer calls: forward output on sampled tokens that the oracle
    # evaluates one by one (with the GPU's routing), and the norm's saved statistics for every token
    w = synth.c3()
    t = synth.generate(w)
    t["x"] = synth.round_to_bf16(t["x"] * 1.5)
    wn = norm_weight(w)
    gpu = gpu_layer(w, t, wn)
    assert gpu["status"] == 0
    xn64, inv64 = orc.rmsnorm(t["x"], wn, EPS)
    assert helpers.rel_err(gpu["inv_rms"], inv64) < 1e-5
    assert helpers.rel_err(gpu["xn"], xn64) < 2e-2
    params = synth.params_of(t)
    xn_r = synth.round_to_bf16(xn64)
    rng = np.random.default_rng(1)
    toks = np.unique(np.concatenate([rng.integers(0, w.tokens, 16), [0, w.tokens - 1]]))
    ref = np.stack([t["x"][i] + orc.token_forward(xn_r[i], params, w.top_k, w.lora_alpha,
                                                  forced_experts=gpu["expert_idx"][i])[0] for i in toks])
    err = np.abs(gpu["h"][toks] - ref).max() / np.abs(ref).max()
    assert err < 2e-2, f"sampled h error {err:.3e}"


def test_layer_7b_shape_2048_tokens_every_gradient():
    # the layer calls at the 7B shape: every output and every gradient (the norm's Jacobian and the residual path
    # included) against the oracle's layer_forward / layer_backward
    w = synth.c3().with_(name="C3-layer-2048", tokens=2048)
    t = synth.generate(w)
    t["x"] = synth.round_to_bf16(t["x"] * 1.5 + 0.05)
    wn = norm_weight(w)
    gpu = gpu_layer(w, t, wn)
    errs = compare(w, gpu, oracle_layer(w, t, wn, gpu), 2e-2)
    print("layer, 7B shape, 2048 tokens:", {n: f"{v:.2e}" for n, v in errs.items()})
