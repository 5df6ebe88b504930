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
