"""Parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times (bf16, tensor-core path).

Where a whole oracle pass is affordable (the 7B-shaped training step, reduced-token passes of the
13B shape and of the skew sweep) every output is compared.  Where it is not (32768 tokens), the
routing and the permutation are still compared for every token and the outputs on sampled tokens
the oracle evaluates one by one."""
import numpy as np
import pytest

import helpers
from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def sampled_forward_check(w, n_samples=24, seed=0):
    t = synth.generate(w, with_dy=True)
    gpu = helpers.gpu_run(w, t, backward=False)
    assert gpu["status"] == 0
    params = synth.params_of(t)
    route = orc.router_forward(t["x"], params["w_router"], params["router_bias"], w.top_k)
    clear = route["margin"] > 2e-4
    np.testing.assert_array_equal(gpu["expert_idx"][clear], route["expert_idx"][clear])
    # permutation of the GPU's own routing must be the canonical one (bit-exact integer work)
    disp = orc.dispatch(gpu["expert_idx"], w.n_experts)
    np.testing.assert_array_equal(gpu["perm"], disp["perm"])
    np.testing.assert_array_equal(gpu["seg_off"], disp["seg_off"])
    assert helpers.rel_err(gpu["probs"], route["probs"]) < 1e-5
    rng = np.random.default_rng(seed)
    toks = np.unique(np.concatenate([rng.integers(0, w.tokens, n_samples), [0, w.tokens - 1]]))
    ref = np.stack([orc.token_forward(t["x"][i], params, w.top_k, w.lora_alpha, forced_experts=gpu["expert_idx"][i])[0]
                    for i in toks])
    scale = np.abs(ref).max()
    err = np.abs(gpu["y"][toks] - ref).max() / scale
    assert err < TOL_BF16, f"{w.name}: sampled y error {err:.3e}"
    shares = np.diff(gpu["seg_off"]) / (w.tokens * w.top_k)
    return shares


def full_check(w, **kw):
    t = synth.generate(w)
    gpu = helpers.gpu_run(w, t, **kw)
    ref = helpers.oracle_run(w, t, gpu, **{k: v for k, v in kw.items() if k in ("aux_coef", "want_dx")})
    return helpers.check_parity(w, gpu, ref, TOL_BF16, want_dx=kw.get("want_dx", True))


def test_c2_forward_full_size_sampled_tokens():
    sampled_forward_check(synth.c2())


def test_c3_training_step_full_size_every_output():
    errs = full_check(synth.c3(), aux_coef=0.01)
    print("C3 relative errors:", {k: f"{v:.2e}" for k, v in errs.items()})


def test_c4_13b_shape_sampled_forward_at_8192_and_full_check_at_2048_tokens():
    sampled_forward_check(synth.c4(), n_samples=12)
    full_check(synth.c4().with_(name="C4-2048", tokens=2048), aux_coef=0.01)


@pytest.mark.parametrize("make", [synth.llama3_8b, synth.wide_2b])
def test_second_workload_shapes_sampled_forward_at_4096_and_full_check_at_1024_tokens(make):
    sampled_forward_check(make(4096), n_samples=12)
    full_check(make(1024), aux_coef=0.01)


@pytest.mark.parametrize("N,k,r", [(8, 1, 8), (8, 2, 16), (8, 2, 64), (16, 1, 16), (16, 2, 8), (16, 2, 64)])
def test_c5_skew_sweep_512_tokens(N, k, r):
    w = synth.c5(N, k, r, 512)
    full_check(w, aux_coef=0.01)


def test_c5_skew_sweep_4096_tokens_largest_rank():
    w = synth.c5(16, 2, 64, 4096)
    t = synth.generate(w)
    gpu = helpers.gpu_run(w, t, aux_coef=0.01)
    ref = helpers.oracle_run(w, t, gpu, aux_coef=0.01)
    helpers.check_parity(w, gpu, ref, TOL_BF16)
    shares = np.sort(np.diff(gpu["seg_off"]) / (w.tokens * w.top_k))[::-1]
    print("achieved slot shares, N=16 k=2:", np.round(shares, 3))
    assert shares[0] > 2.5 * shares[-1]          # the bias does skew the load


def test_c5_32768_tokens_routing_exact_and_sampled_outputs():
    shares = sampled_forward_check(synth.c5(8, 2, 16, 32768), n_samples=12)
    print("achieved slot shares, N=8 k=2:", np.round(np.sort(shares)[::-1], 3))
