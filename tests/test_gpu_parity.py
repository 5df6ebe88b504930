"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on
the same seeded tensors.  Routing must be bit-exact on tokens with a clear margin; values
must agree to 1e-4 of the tensor's largest reference value in fp32 mode and 2e-2 in bf16 mode."""
import numpy as np
import pytest

import helpers
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4
TOL_BF16 = 2e-2


def small(name, dtype="bf16", **kw):
    base = dict(tokens=300, d_model=256, d_ff=688, n_experts=8, top_k=2, rank=16, lora_alpha=32.0, dtype=dtype,
                std_frozen=0.05, std_a=0.06, std_b=0.05, seed=synth.BASE_SEED + 100)
    base.update(kw)
    return synth.Workload(name, **base)


def run_case(w, tol, **kw):
    t = synth.generate(w)
    gpu = helpers.gpu_run(w, t, **kw)
    okw = {k: v for k, v in kw.items() if k in ("backward", "want_dx", "aux_coef", "aux_f_mode")}
    if "renormalize" in kw:
        okw["renormalize"] = bool(kw["renormalize"])
    ref = helpers.oracle_run(w, t, gpu, **okw)
    return helpers.check_parity(w, gpu, ref, tol, backward=kw.get("backward", True), want_dx=kw.get("want_dx", True))


def test_c1_tiny_fp32_forward_backward_aux():
    run_case(synth.c1(), TOL_FP32, aux_coef=0.01)


@pytest.mark.parametrize("T", [1, 7, 128, 129, 300, 1000])
def test_fp32_ragged_token_counts(T):
    run_case(small(f"fp32-T{T}", "fp32", tokens=T, rank=8, n_experts=4), TOL_FP32)


@pytest.mark.parametrize("N,k,r", [(1, 1, 8), (4, 1, 8), (4, 4, 8), (8, 2, 16), (16, 2, 64), (32, 8, 8), (16, 1, 128)])
def test_bf16_expert_topk_rank_grid(N, k, r):
    run_case(small(f"bf16-N{N}-k{k}-r{r}", n_experts=N, top_k=k, rank=r, lora_alpha=2.0 * r, std_a=1.0 / r), TOL_BF16)


@pytest.mark.parametrize("N,k,r", [(4, 2, 4), (8, 3, 12), (5, 2, 8)])
def test_fp32_odd_sizes(N, k, r):
    run_case(small(f"fp32-N{N}-k{k}-r{r}", "fp32", n_experts=N, top_k=k, rank=r, tokens=211, d_ff=200, d_model=72),
             TOL_FP32)


def test_bf16_llama_like_small_slice():
    # several 128-row tiles per expert, a ragged tail, f not a multiple of 128
    run_case(small("bf16-slice", tokens=1111, d_model=512, d_ff=1376, std_frozen=0.02, std_a=1.0 / 16, std_b=0.01),
             TOL_BF16)


def test_without_dx_and_without_backward():
    run_case(small("no-dx"), TOL_BF16, want_dx=False)
    run_case(small("fwd-only"), TOL_BF16, backward=False)


def test_unrenormalised_gates_and_all_selection_counting():
    run_case(small("no-renorm", "fp32", rank=8), TOL_FP32, renormalize=0)
    run_case(small("f-mode-1", "fp32", rank=8), TOL_FP32, aux_f_mode=1)


def test_skewed_routing_with_empty_experts():
    w = small("skew", "fp32", n_experts=8, rank=8, zipf_s=1.2)
    t = synth.generate(w)
    t["router_bias"] = np.array([3, 2, 1, 0, -30, -30, -1, -30], np.float32)   # three experts never chosen
    gpu = helpers.gpu_run(w, t)
    ref = helpers.oracle_run(w, t, gpu)
    helpers.check_parity(w, gpu, ref, TOL_FP32)
    counts = np.diff(gpu["seg_off"])
    assert counts[4] == 0 and counts[5] == 0 and counts[7] == 0 and counts.sum() == w.tokens * w.top_k
    for n in ("d_a_gate", "d_b_gate", "d_a_down", "d_b_down"):
        assert np.all(gpu[n][4] == 0) and np.all(gpu[n][7] == 0)


def test_zero_tokens_is_a_no_op():
    w = small("empty", tokens=0)
    t = synth.generate(w)
    gpu = helpers.gpu_run(w, t)
    assert gpu["status"] == 0 and gpu["loss"] == 0.0
    for n in helpers.GRAD_NAMES:
        assert np.all(gpu[n] == 0)


def test_exact_ties_follow_the_lower_index_rule_and_are_flagged():
    w = small("ties", "fp32", rank=8, n_experts=4)
    t = synth.generate(w)
    t["w_router"][:] = t["w_router"][0]          # all logits equal for every token
    gpu = helpers.gpu_run(w, t, backward=False)
    assert (gpu["expert_idx"] == np.array([0, 1])).all()
    assert (gpu["low_margin"] == 1).all()
    np.testing.assert_allclose(gpu["gates"], 0.5, rtol=1e-6)


def test_gradient_accumulation_adds_to_the_outputs():
    w = small("accum", "fp32", rank=8, n_experts=4)
    t = synth.generate(w)
    base = helpers.gpu_run(w, t)
    init = {n: np.full_like(base[n], 0.5) for n in helpers.GRAD_NAMES}
    acc = helpers.gpu_run(w, t, accumulate=1, grads_init=init)
    for n in helpers.GRAD_NAMES:
        np.testing.assert_allclose(acc[n], base[n] + 0.5, rtol=1e-5, atol=1e-6)


def test_two_calls_in_a_row_are_bit_identical():
    w = small("repeat")
    t = synth.generate(w)
    a = helpers.gpu_run(w, t)
    b = helpers.gpu_run(w, t, repeats=2)
    for n in ("y", "d_x") + helpers.GRAD_NAMES:
        np.testing.assert_array_equal(a[n], b[n])


def test_identity_zero_B_reproduces_the_frozen_ffn_on_the_gpu():
    w = small("zero-b", "fp32", rank=8)
    t = synth.generate(w)
    for n in ("b_gate", "b_up", "b_down"):
        t[n][:] = 0
    gpu = helpers.gpu_run(w, t, backward=False)
    x = t["x"].astype(np.float64)
    a = x @ t["w_gate"].astype(np.float64).T
    ref = (a / (1 + np.exp(-a)) * (x @ t["w_up"].astype(np.float64).T)) @ t["w_down"].astype(np.float64).T
    assert helpers.rel_err(gpu["y"], ref) < TOL_FP32


@pytest.mark.parametrize("r", [24, 48, 96])
def test_bf16_ranks_between_the_native_operand_widths(r):
    # ranks that are multiples of 8 but not 8, 16, 32, 64 or 128: the grouped kernels work on operands zero-padded
    # to the next of those widths
    run_case(small(f"bf16-r{r}", n_experts=4, top_k=2, rank=r, lora_alpha=2.0 * r, std_a=1.0 / r, tokens=517, d_ff=1000),
             TOL_BF16)


def test_non_finite_logits_never_become_repeated_or_invalid_indices():
    # one token whose x row is NaN, and a bias that masks all but one expert for everybody: the k choices must stay
    # distinct and the permutation complete (the workspace comes uncleared from the allocator); NaN may show up in
    # values only
    w = small("nonfinite", "bf16", n_experts=8, top_k=2, rank=16, tokens=700)
    t = synth.generate(w)
    t["x"][123, :] = np.nan
    t["router_bias"] = np.full(8, -np.inf, np.float32)
    t["router_bias"][5] = 0.0
    gpu = helpers.gpu_run(w, t, backward=True)
    assert gpu["status"] == 0
    idx = gpu["expert_idx"]
    assert idx.min() >= 0 and idx.max() < 8
    assert (idx[:, 0] != idx[:, 1]).all()
    keep = np.arange(w.tokens) != 123
    assert (idx[keep, 0] == 5).all()                                       # the one finite logit wins
    assert sorted(gpu["perm"].tolist()) == list(range(w.tokens * w.top_k))
    counts = np.diff(gpu["seg_off"])
    assert counts.sum() == w.tokens * w.top_k and (counts >= 0).all()
    assert np.isnan(gpu["y"][123]).all()
    ok = np.ones(w.tokens, bool)
    ok[123] = False
    assert np.isfinite(gpu["y"][ok]).all()                                 # gates are (1, 0): exp(-inf) = 0


def test_a_bounded_wait_that_runs_out_is_reported_as_a_status_and_the_context_stays_usable():
    import torch
    from paper_2404_15159_b200 import binding as B

    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert B.mixlora_device_status(ws) == 0
    B.mixlora_selftest_wait_timeout(ws, 1 << 10)
    assert B.mixlora_device_status(ws) == 5                                # MIXLORA_ERR_DEVICE_TIMEOUT
    assert "wait" in B.status_string(5)
    run_case(small("after-timeout", "fp32", rank=8, n_experts=4, tokens=64), TOL_FP32)   # the device still works


def test_the_serial_option_changes_scheduling_only():
    from paper_2404_15159_b200 import binding as B

    w = small("serial")
    t = synth.generate(w)
    a = helpers.gpu_run(w, t)
    B.mixlora_set_option(B.MIXLORA_OPT_SERIAL, 1)
    try:
        b = helpers.gpu_run(w, t)
    finally:
        B.mixlora_set_option(B.MIXLORA_OPT_SERIAL, 0)
    for n in ("y", "d_x") + helpers.GRAD_NAMES:
        np.testing.assert_array_equal(a[n], b[n])
    with pytest.raises(B.MixLoraError):
        B.mixlora_set_option(77, 1)


@pytest.mark.parametrize("f_mode", [0, 1])
def test_auxiliary_loss_of_the_whole_batch_over_two_shards(f_mode):
    # Eq. 8-9 are fractions of the whole batch.  Two shards run one after the other on this GPU: forward, the
    # un-normalised sums of each, their total handed back with the batch's token count, backward.  The loss must be
    # the full batch's and the shards' gradients must add up to the oracle's full-batch gradients.
    import torch
    from oracle import mixlora_oracle as orc
    from paper_2404_15159_b200 import binding as B

    w = small("aux-global", "fp32", rank=8, n_experts=4, tokens=300)
    coef = 0.5
    t = synth.generate(w)
    params_np = synth.params_of(t)
    dev = {n: (None if v is None else torch.from_numpy(np.ascontiguousarray(v, np.float32)).cuda()) for n, v in t.items()}
    cuts = [(0, 113), (113, 300)]
    state = []
    psum = torch.zeros(w.n_experts, device="cuda")
    cnt = torch.zeros(w.n_experts, device="cuda")
    loss_local = torch.zeros(1, device="cuda")
    for b, e in cuts:
        shape = B.make_shape(e - b, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha,
                             B.MIXLORA_DTYPE_FP32, 1, f_mode)
        params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"][b:e])
        ws = B.alloc_workspace(shape, True)
        y = torch.empty(e - b, w.d_model, device="cuda")
        B.mixlora_ffn_forward(shape, params, y, ws)
        ps, c = torch.empty(w.n_experts, device="cuda"), torch.empty(w.n_experts, device="cuda")
        B.mixlora_aux_stats(shape, ws, ps, c)
        if b == 0:      # the shard's own loss, before the batch's F and P replace the shard's in its workspace
            B.mixlora_aux_loss(shape, ws, coef, loss_local)
        psum += ps
        cnt += c
        state.append((shape, params, ws, y))
    torch.cuda.synchronize()
    # the oracle on the whole batch; a token whose deciding logit gap is below the flag threshold may keep the
    # library's choice when that choice is one the near tie allows
    gpu_idx = np.concatenate([B.mixlora_routing_view(st[0], st[2])["expert_idx"].cpu().numpy() for st in state])
    y_ref, saved = orc.ffn_forward(t["x"], params_np, w.top_k, w.lora_alpha)
    route = saved["route"]
    diff = (gpu_idx != route["expert_idx"]).any(axis=1)
    assert not (diff & (route["margin"] >= helpers.ROUTE_MARGIN)).any()
    if diff.any():
        helpers.assert_near_tie(route["logits"], route["expert_idx"], gpu_idx, diff, helpers.ROUTE_MARGIN)
        y_ref, saved = orc.ffn_forward(t["x"], params_np, w.top_k, w.lora_alpha, forced_expert_idx=gpu_idx)
    loss_ref, F_ref, P_ref = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], coef, f_mode)
    g_ref = orc.ffn_backward(t["x"], params_np, t["dy"], saved, aux_coef=coef, aux_f_mode=f_mode)
    total = {n: None for n in helpers.GRAD_NAMES}
    dx = np.zeros_like(t["x"], dtype=np.float32)
    for (b, e), (shape, params, ws, y) in zip(cuts, state):
        loss = torch.zeros(1, device="cuda")
        F, P = torch.zeros(w.n_experts, device="cuda"), torch.zeros(w.n_experts, device="cuda")
        B.mixlora_aux_loss_global(shape, ws, coef, psum, cnt, w.tokens, loss, F, P)
        g = {n: torch.full(tuple(np.shape(g_ref[n])), float("nan"), device="cuda") for n in helpers.GRAD_NAMES}
        g["d_x"] = torch.empty(e - b, w.d_model, device="cuda")
        B.mixlora_ffn_backward(shape, params, dev["dy"][b:e], coef, ws, B.make_grads(**g))
        torch.cuda.synchronize()
        assert B.mixlora_device_status(ws) == 0
        assert abs(float(loss.item()) - loss_ref) <= 1e-5 * abs(loss_ref)
        assert helpers.rel_err(F.cpu().numpy(), F_ref) < 1e-6 and helpers.rel_err(P.cpu().numpy(), P_ref) < 1e-5
        for n in helpers.GRAD_NAMES:
            v = g[n].cpu().numpy().astype(np.float64)
            total[n] = v if total[n] is None else total[n] + v
        dx[b:e] = g["d_x"].cpu().numpy()
    for n in helpers.GRAD_NAMES:
        assert helpers.rel_err(total[n], g_ref[n]) <= TOL_FP32, n
    assert helpers.rel_err(dx, g_ref["d_x"]) <= TOL_FP32
    # and a per-shard loss (no exchange) is a different number: the exchange matters
    assert abs(float(loss_local.item()) - loss_ref) > 1e-4 * abs(loss_ref)
