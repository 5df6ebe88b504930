"""Plain LoRA on a linear layer (Eq. 1; the attention projections of a MixLoRA model) through the C ABI against
the CPU oracle: forward, input gradient, LoRA gradients, accumulation, ragged and empty token counts."""
import numpy as np
import pytest

import helpers
from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu


def make(T, d_in, d_out, r, seed, bf16):
    rng = np.random.default_rng(seed)
    rnd = synth.round_to_bf16 if bf16 else (lambda v: np.asarray(v, np.float32).astype(np.float64))
    return dict(x=rnd(rng.standard_normal((T, d_in))), w=rnd(rng.standard_normal((d_out, d_in)) * 0.03),
                a=rnd(rng.standard_normal((r, d_in)) / r), b=rnd(rng.standard_normal((d_out, r)) * 0.05),
                dy=rnd(rng.standard_normal((T, d_out))))


def run_gpu(t, T, d_in, d_out, r, alpha, bf16, accumulate=False):
    import torch
    from paper_2404_15159_b200 import binding as B

    act = torch.bfloat16 if bf16 else torch.float32
    dev = {n: torch.from_numpy(np.ascontiguousarray(v)).cuda().to(act) if v.size else torch.empty(8, dtype=act, device="cuda")
           for n, v in t.items()}
    shape = B.make_linear_shape(T, d_in, d_out, r, alpha, B.MIXLORA_DTYPE_BF16 if bf16 else B.MIXLORA_DTYPE_FP32)
    ws = B.alloc_linear_workspace(shape)
    y = torch.full((max(T, 1), d_out), float("nan"), dtype=act, device="cuda")
    d_x = torch.full((max(T, 1), d_in), float("nan"), dtype=act, device="cuda")
    init = 0.5 if accumulate else float("nan")
    d_a = torch.full((r, d_in), init, dtype=torch.float32, device="cuda")
    d_b = torch.full((d_out, r), init, dtype=torch.float32, device="cuda")
    B.mixlora_lora_linear_forward(shape, dev["x"], dev["w"], dev["a"], dev["b"], y, ws)
    B.mixlora_lora_linear_backward(shape, dev["x"], dev["w"], dev["a"], dev["b"], dev["dy"], ws, d_a, d_b, d_x,
                                   accumulate=1 if accumulate else 0)
    torch.cuda.synchronize()
    assert B.mixlora_lora_linear_status(ws) == 0
    return dict(y=y[:T].float().cpu().numpy(), d_x=d_x[:T].float().cpu().numpy(), d_a=d_a.cpu().numpy(),
                d_b=d_b.cpu().numpy())


@pytest.mark.parametrize("T,d_in,d_out,r,bf16", [(300, 256, 512, 8, False), (1000, 512, 512, 16, True),
                                                 (257, 1024, 384, 64, True), (4096, 4096, 4096, 16, True)])
def test_lora_linear_matches_the_oracle(T, d_in, d_out, r, bf16):
    alpha = 2.0 * r
    t = make(T, d_in, d_out, r, 900 + T, bf16)
    gpu = run_gpu(t, T, d_in, d_out, r, alpha, bf16)
    ref = dict(y=orc.lora_linear_forward(t["x"], t["w"], t["a"], t["b"], alpha),
               **orc.lora_linear_backward(t["x"], t["w"], t["a"], t["b"], alpha, t["dy"]))
    tol = 2e-2 if bf16 else 1e-4
    for n in ("y", "d_x", "d_a", "d_b"):
        e = helpers.rel_err(gpu[n], ref[n])
        assert e <= tol, f"{n}: relative error {e:.3e} > {tol:.1e}"


def test_lora_linear_accumulates_and_handles_no_tokens():
    T, d_in, d_out, r, alpha = 200, 256, 256, 16, 32.0
    t = make(T, d_in, d_out, r, 77, True)
    plain = run_gpu(t, T, d_in, d_out, r, alpha, True)
    acc = run_gpu(t, T, d_in, d_out, r, alpha, True, accumulate=True)
    np.testing.assert_allclose(acc["d_a"], plain["d_a"] + 0.5, rtol=0, atol=1e-5 * np.abs(plain["d_a"]).max() + 1e-6)
    np.testing.assert_allclose(acc["d_b"], plain["d_b"] + 0.5, rtol=0, atol=1e-5 * np.abs(plain["d_b"]).max() + 1e-6)
    empty = make(0, d_in, d_out, r, 78, True)
    out = run_gpu(empty, 0, d_in, d_out, r, alpha, True)
    assert not out["d_a"].any() and not out["d_b"].any()
