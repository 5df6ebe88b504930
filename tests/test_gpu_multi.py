"""Multi-model calls (Section 3.3 (II)): several adapters sharing one frozen FFN in a single call must give, for
every adapter, exactly the results of the single-model calls, and those match the CPU oracle."""
import numpy as np
import pytest

import helpers
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu

GRADS = helpers.GRAD_NAMES


def adapters():
    base = dict(d_model=512, d_ff=1408, lora_alpha=32.0, dtype="bf16", std_frozen=0.03, std_a=0.06, std_b=0.03)
    return [synth.Workload("multi-a", tokens=700, n_experts=8, top_k=2, rank=16, seed=synth.BASE_SEED + 400, **base),
            synth.Workload("multi-b", tokens=333, n_experts=4, top_k=1, rank=8, seed=synth.BASE_SEED + 401, **base),
            synth.Workload("multi-c", tokens=1030, n_experts=16, top_k=3, rank=32, seed=synth.BASE_SEED + 402, **base)]


def test_three_adapters_one_frozen_ffn_equal_the_single_model_calls():
    import torch
    from paper_2404_15159_b200 import binding as B

    ws_ = adapters()
    tens = [synth.generate(w) for w in ws_]
    for t in tens[1:]:                                   # one frozen FFN for all adapters
        for n in ("w_gate", "w_up", "w_down"):
            t[n] = tens[0][n]
    act = torch.bfloat16
    frozen = {n: torch.from_numpy(tens[0][n]).cuda().to(act) for n in ("w_gate", "w_up", "w_down")}
    shapes, params, ys, wss, dys, grads, gbufs = [], [], [], [], [], [], []
    keep = []
    for w, t in zip(ws_, tens):
        dev = dict(frozen)
        for n, v in t.items():
            if n in frozen or v is None:
                dev.setdefault(n, None)
                continue
            dev[n] = torch.from_numpy(v).cuda() if n in ("w_router", "router_bias") else torch.from_numpy(v).cuda().to(act)
        keep.append(dev)
        shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha)
        shapes.append(shape)
        params.append(B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"]))
        ys.append(torch.empty(w.tokens, w.d_model, dtype=act, device="cuda"))
        wss.append(B.alloc_workspace(shape, True))
        dys.append(dev["dy"])
        g = {n: torch.full(tuple(t[n[2:]].shape) if n != "d_router_bias" else (w.n_experts,), float("nan"),
                           dtype=torch.float32, device="cuda") for n in GRADS}
        g["d_x"] = torch.full((w.tokens, w.d_model), float("nan"), dtype=act, device="cuda")
        gbufs.append(g)
        grads.append(B.make_grads(**g))
    coefs = [0.01, 0.0, 0.02]
    B.mixlora_multi_ffn_forward(shapes, params, ys, wss)
    B.mixlora_multi_ffn_backward(shapes, params, dys, coefs, wss, grads)
    torch.cuda.synchronize()
    for i, (w, t) in enumerate(zip(ws_, tens)):
        assert B.mixlora_device_status(wss[i]) == 0
        single = helpers.gpu_run(w, t, aux_coef=coefs[i])
        np.testing.assert_array_equal(ys[i].float().cpu().numpy(), single["y"])
        for n in GRADS + ("d_x",):
            np.testing.assert_array_equal(gbufs[i][n].float().cpu().numpy(), single[n], err_msg=f"{w.name} {n}")
        ref = helpers.oracle_run(w, t, single, aux_coef=coefs[i])
        helpers.check_parity(w, single, ref, 2e-2)


def test_multi_call_rejects_adapters_with_different_frozen_weights():
    import torch
    from paper_2404_15159_b200 import binding as B

    w = adapters()[1]
    t = synth.generate(w)
    act = torch.bfloat16
    dev = {n: (None if v is None else (torch.from_numpy(v).cuda() if n in ("w_router", "router_bias")
                                      else torch.from_numpy(v).cuda().to(act))) for n, v in t.items()}
    other = dict(dev)
    other["w_up"] = dev["w_up"].clone()                  # same values, different buffer: not shared
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha)
    ps = [B.make_params(**{n: dd[n] for n in synth.PARAM_NAMES}, x=dd["x"]) for dd in (dev, other)]
    ys = [torch.empty(w.tokens, w.d_model, dtype=act, device="cuda") for _ in range(2)]
    wss = [B.alloc_workspace(shape, False) for _ in range(2)]
    with pytest.raises(B.MixLoraError) as err:
        B.mixlora_multi_ffn_forward([shape, shape], ps, ys, wss)
    assert err.value.status == 1


def test_backward_overlap_signals_after_the_parameter_gradients_and_changes_no_result():
    # data-parallel replicas all-reduce the LoRA / router gradients while the input-gradient product still runs:
    # what a second stream reads at the signal must already be the final gradients
    w = adapters()[0]
    t = synth.generate(w)
    plain = helpers.gpu_run(w, t, aux_coef=0.01)
    over = helpers.gpu_run(w, t, aux_coef=0.01, overlap=True)
    assert over["status"] == 0
    for n in GRADS:
        np.testing.assert_array_equal(over[n], plain[n])
        np.testing.assert_array_equal(over["snap_" + n], plain[n])
    np.testing.assert_array_equal(over["d_x"], plain["d_x"])

