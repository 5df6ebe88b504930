"""Pins of the MixDoRA oracle (CPU only).  The paper names MixDoRA (Section 4.1, Table 1) without a formula, so
what fixes the oracle is what the weight-decomposed form must reduce to: MixLoRA when the magnitudes equal the
norms, the frozen FFN when B = 0 and the magnitudes are the row norms of W, a dense FFN with explicitly merged
weights for N = 1, homogeneity in the magnitudes, and central differences with the norms held constant."""
import numpy as np
import pytest

from oracle import mixdora_oracle as dora
from oracle import mixlora_oracle as orc


def tiny(seed=0, T=7, d=8, f=12, N=3, k=2, r=2, bias=False):
    rng = np.random.default_rng(seed)
    p = dict(w_gate=rng.normal(0, 0.5, (f, d)), w_up=rng.normal(0, 0.5, (f, d)), w_down=rng.normal(0, 0.5, (d, f)),
             w_router=rng.normal(0, 1.0, (N, d)), router_bias=rng.normal(0, 0.3, N) if bias else None,
             a_gate=rng.normal(0, 0.5, (N, r, d)), b_gate=rng.normal(0, 0.5, (N, f, r)),
             a_up=rng.normal(0, 0.5, (N, r, d)), b_up=rng.normal(0, 0.5, (N, f, r)),
             a_down=rng.normal(0, 0.5, (N, r, f)), b_down=rng.normal(0, 0.5, (N, d, r)))
    m = dict(gate=rng.uniform(0.5, 1.5, (N, f)), up=rng.uniform(0.5, 1.5, (N, f)), down=rng.uniform(0.5, 1.5, (N, d)))
    x = rng.normal(0, 1, (T, d))
    dy = rng.normal(0, 1, (T, d))
    return x, p, m, dy, k, 2.0 * r


def test_magnitudes_equal_to_the_norms_give_mixlora_exactly():
    x, p, m, dy, k, alpha = tiny(1)
    n = dora.all_norms(p, alpha)
    y, _ = dora.ffn_forward(x, p, n, k, alpha)
    y_ref, _ = orc.ffn_forward(x, p, k, alpha)
    np.testing.assert_allclose(y, y_ref, rtol=1e-12, atol=1e-12)
    # ... and other magnitudes do not
    y2, _ = dora.ffn_forward(x, p, m, k, alpha)
    assert np.abs(y2 - y_ref).max() > 1e-3


def test_zero_b_with_row_norm_magnitudes_is_the_frozen_ffn():
    x, p, m, dy, k, alpha = tiny(2)
    for n in ("b_gate", "b_up", "b_down"):
        p[n] = np.zeros_like(p[n])
    N = p["a_gate"].shape[0]
    mag = dict(gate=np.tile(np.linalg.norm(p["w_gate"], axis=1), (N, 1)),
               up=np.tile(np.linalg.norm(p["w_up"], axis=1), (N, 1)),
               down=np.tile(np.linalg.norm(p["w_down"], axis=1), (N, 1)))
    y, _ = dora.ffn_forward(x, p, mag, k, alpha)
    a = x @ p["w_gate"].T
    ref = (a / (1 + np.exp(-a)) * (x @ p["w_up"].T)) @ p["w_down"].T
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-12)


def test_single_expert_is_a_dense_ffn_with_the_three_merged_dora_weights():
    x, p, m, dy, k, alpha = tiny(3, N=1, k=1)
    y, _ = dora.ffn_forward(x, p, m, 1, alpha)
    s = alpha / p["a_gate"].shape[1]

    def merged(w, a, b, mag):          # retyped from the definition: scale every output row of W + s B A to length mag
        full = w + s * b @ a
        return full * (mag / np.linalg.norm(full, axis=1))[:, None]

    w1 = merged(p["w_gate"], p["a_gate"][0], p["b_gate"][0], m["gate"][0])
    w3 = merged(p["w_up"], p["a_up"][0], p["b_up"][0], m["up"][0])
    w2 = merged(p["w_down"], p["a_down"][0], p["b_down"][0], m["down"][0])
    np.testing.assert_allclose(np.linalg.norm(w1, axis=1), m["gate"][0], rtol=1e-12)   # rows have length m
    a = x @ w1.T
    ref = (a / (1 + np.exp(-a)) * (x @ w3.T)) @ w2.T
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-12)


def test_shared_projection_form_equals_the_token_by_token_definition():
    x, p, m, dy, k, alpha = tiny(4, bias=True)
    y, _ = dora.ffn_forward(x, p, m, k, alpha)
    np.testing.assert_allclose(y, dora.ffn_forward_merged(x, p, m, k, alpha), rtol=1e-11, atol=1e-12)


def test_norms_match_the_expanded_square():
    # ||W_o + s B_o A||^2 = ||W_o||^2 + 2 s B_o . (W A^T)_o + s^2 B_o (A A^T) B_o^T
    x, p, m, dy, k, alpha = tiny(5)
    s = alpha / p["a_gate"].shape[1]
    n = dora.all_norms(p, alpha)
    for name, w, a, b in (("gate", p["w_gate"], p["a_gate"], p["b_gate"]), ("down", p["w_down"], p["a_down"], p["b_down"])):
        for e in range(a.shape[0]):
            sq = (w * w).sum(1) + 2 * s * np.einsum("or,or->o", b[e], w @ a[e].T) \
                + s * s * np.einsum("or,rq,oq->o", b[e], a[e] @ a[e].T, b[e])
            np.testing.assert_allclose(n[name][e] ** 2, sq, rtol=1e-12)


def test_output_is_homogeneous_in_the_down_magnitude_and_the_up_magnitude():
    x, p, m, dy, k, alpha = tiny(6)
    y, _ = dora.ffn_forward(x, p, m, k, alpha)
    m2 = dict(m, down=3.0 * m["down"])
    y2, _ = dora.ffn_forward(x, p, m2, k, alpha)
    np.testing.assert_allclose(y2, 3.0 * y, rtol=1e-12)
    m3 = dict(m, up=0.5 * m["up"])                      # b enters h linearly, h enters o linearly
    y3, _ = dora.ffn_forward(x, p, m3, k, alpha)
    np.testing.assert_allclose(y3, 0.5 * y, rtol=1e-12)


def loss(x, p, m, dy, k, alpha, aux, norms):
    y, saved = dora.ffn_forward(x, p, m, k, alpha, norms=norms)
    la, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], aux, 0)
    return float(np.sum(dy * y) + la)


@pytest.mark.parametrize("k,aux", [(2, 0.0), (2, 0.3), (3, 0.3)])
def test_central_differences_with_the_norms_held_constant(k, aux):
    x, p, m, dy, _, alpha = tiny(7, k=k, bias=True)
    norms = dora.all_norms(p, alpha)
    y, saved = dora.ffn_forward(x, p, m, k, alpha)
    assert saved["route"]["margin"].min() > 1e-3 or k == 3
    g = dora.ffn_backward(x, p, m, dy, saved, aux_coef=aux)
    h = 1e-6
    rng = np.random.default_rng(11)

    def check(getter, grad, n_probe=6):
        arr = getter()
        for _ in range(n_probe):
            i = tuple(int(rng.integers(0, sdim)) for sdim in arr.shape)
            old = arr[i]
            arr[i] = old + h
            lp = loss(x, p, m, dy, k, alpha, aux, norms)
            arr[i] = old - h
            lm = loss(x, p, m, dy, k, alpha, aux, norms)
            arr[i] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grad[i]) <= 1e-6 * max(1.0, abs(fd)), (i, fd, grad[i])

    for n in ("a_gate", "b_gate", "a_up", "b_up", "a_down", "b_down", "w_router", "router_bias"):
        check(lambda n=n: p[n], g["d_" + n])
    for n in ("gate", "up", "down"):
        check(lambda n=n: m[n], g["d_m_" + n])
    check(lambda: x, g["d_x"])


def test_the_norm_really_is_outside_the_gradient():
    # differences that let the norm move with B give another number: the analytic gradient is the detached one
    x, p, m, dy, k, alpha = tiny(8)
    y, saved = dora.ffn_forward(x, p, m, k, alpha)
    g = dora.ffn_backward(x, p, m, dy, saved)
    h = 1e-6
    i = (0, 1, 0)
    old = p["b_gate"][i]
    p["b_gate"][i] = old + h
    lp = loss(x, p, m, dy, k, alpha, 0.0, None)
    p["b_gate"][i] = old - h
    lm = loss(x, p, m, dy, k, alpha, 0.0, None)
    p["b_gate"][i] = old
    moving = (lp - lm) / (2 * h)
    assert abs(moving - g["d_b_gate"][i]) > 1e-4 * max(1.0, abs(moving))


def test_a_planted_mistake_in_the_magnitude_gradient_is_caught():
    x, p, m, dy, k, alpha = tiny(9)
    norms = dora.all_norms(p, alpha)
    y, saved = dora.ffn_forward(x, p, m, k, alpha)
    g = dora.ffn_backward(x, p, m, dy, saved)
    wrong = g["d_m_gate"] * norms["gate"] / m["gate"]       # dividing by m instead of n
    h = 1e-6
    i = (1, 3)
    old = m["gate"][i]
    m["gate"][i] = old + h
    lp = loss(x, p, m, dy, k, alpha, 0.0, norms)
    m["gate"][i] = old - h
    lm = loss(x, p, m, dy, k, alpha, 0.0, norms)
    m["gate"][i] = old
    fd = (lp - lm) / (2 * h)
    assert abs(fd - g["d_m_gate"][i]) <= 1e-6 * max(1.0, abs(fd))
    assert abs(fd - wrong[i]) > 1e-3 * max(1.0, abs(fd))
