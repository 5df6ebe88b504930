"""Pins of the CPU oracle against facts the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each one is chosen so that a
plausible slip in the oracle (a dropped term, a wrong sign or index, a
transposed operand, a missing scale) breaks it.
"""
import json
import os

import numpy as np
import pytest
import scipy.special

from oracle import mixlora_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def make_case(T=7, d=10, f=14, N=4, k=2, r=3, alpha=6.0, seed=0, b_scale=0.3, bias=False):
    rng = np.random.default_rng(seed)
    p = dict(
        w_gate=rng.normal(size=(f, d)) * 0.4, w_up=rng.normal(size=(f, d)) * 0.4,
        w_down=rng.normal(size=(d, f)) * 0.4, w_router=rng.normal(size=(N, d)) * 0.5,
        router_bias=(rng.normal(size=N) * 0.2 if bias else None),
        a_gate=rng.normal(size=(N, r, d)) * 0.3, b_gate=rng.normal(size=(N, f, r)) * b_scale,
        a_up=rng.normal(size=(N, r, d)) * 0.3, b_up=rng.normal(size=(N, f, r)) * b_scale,
        a_down=rng.normal(size=(N, r, f)) * 0.3, b_down=rng.normal(size=(N, d, r)) * b_scale,
    )
    x = rng.normal(size=(T, d))
    dy = rng.normal(size=(T, d))
    return x, p, dy, dict(top_k=k, lora_alpha=alpha)


def dense_ffn(x, w1, w3, w2):
    """Textbook SwiGLU FFN, H = W2 (SiLU(W1 x) * W3 x), on whole matrices (Section 3.3)."""
    a = x @ w1.T
    return ((a * scipy.special.expit(a)) * (x @ w3.T)) @ w2.T


# ---- textbook pieces -------------------------------------------------------
def test_softmax_matches_scipy_and_sums_to_one():
    rng = np.random.default_rng(1)
    l = rng.normal(size=(50, 9)) * 5
    p = orc.softmax_rows(l)
    np.testing.assert_allclose(p, scipy.special.softmax(l, axis=1), rtol=1e-13)
    np.testing.assert_allclose(p.sum(1), 1.0, rtol=1e-14)


def test_silu_matches_expit_and_its_derivative_matches_differences():
    v = np.linspace(-8, 8, 401)
    np.testing.assert_allclose(orc.silu(v), v * scipy.special.expit(v), rtol=1e-13, atol=1e-15)
    h = 1e-6
    fd = (orc.silu(v + h) - orc.silu(v - h)) / (2 * h)
    np.testing.assert_allclose(orc.silu_grad(v), fd, atol=1e-8)


def test_router_topk_is_the_k_largest_logits_with_ties_to_lower_index():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(40, 6))
    w = rng.normal(size=(5, 6))
    for k in (1, 2, 3, 5):
        r = orc.router_forward(x, w, None, k)
        for t in range(40):
            l = list(r["logits"][t])
            want = sorted(range(5), key=lambda i: (-l[i], i))[:k]    # brute force
            assert list(r["expert_idx"][t]) == want
        np.testing.assert_allclose(r["gates"].sum(1), 1.0, rtol=1e-14)
        assert (r["gates"] > 0).all() and (r["gates"] <= 1).all()
    # exact ties: identical rows of W give identical logits
    w_tie = np.tile(w[:1], (4, 1))
    r = orc.router_forward(x, w_tie, None, 2)
    assert (r["expert_idx"] == np.array([0, 1])).all()
    assert (r["margin"] == 0).all()


def test_router_gates_equal_softmax_over_selected_logits():
    # Norm(TopK(Softmax(l))) is the softmax restricted to the selected logits
    rng = np.random.default_rng(3)
    x = rng.normal(size=(30, 8)); w = rng.normal(size=(6, 8)); b = rng.normal(size=6)
    r = orc.router_forward(x, w, b, 3)
    sel = np.take_along_axis(x @ w.T + b, r["expert_idx"].astype(np.int64), axis=1)
    np.testing.assert_allclose(r["gates"], scipy.special.softmax(sel, axis=1), rtol=1e-12)
    r2 = orc.router_forward(x, w, b, 3, renormalize=False)
    np.testing.assert_allclose(r2["gates"], np.take_along_axis(r2["probs"], r2["expert_idx"].astype(np.int64), 1))


def test_router_margin_is_the_deciding_logit_gap():
    l = np.array([[3.0, 1.0, 2.5, -1.0]])
    x = np.eye(4)[:1] * 0 + 1.0
    # logits = x @ w.T with x = ones(1,1): use d = 1
    r = orc.router_forward(np.ones((1, 1)), l.T.copy(), None, 2)
    assert list(r["expert_idx"][0]) == [0, 2]
    assert r["margin"][0] == pytest.approx(0.5)          # min(l1-l2 = 0.5, l2-l3 = 1.5)
    r = orc.router_forward(np.ones((1, 1)), l.T.copy(), None, 4)
    assert r["margin"][0] == pytest.approx(0.5)          # only the arg-max gap remains


# ---- dispatch --------------------------------------------------------------
def test_dispatch_is_the_lexicographic_sort_by_expert_then_token():
    rng = np.random.default_rng(4)
    T, N, k = 57, 6, 3
    idx = np.stack([rng.permutation(N)[:k] for _ in range(T)]).astype(np.int32)
    d = orc.dispatch(idx, N)
    slots = [(int(idx[t, j]), t, t * k + j) for t in range(T) for j in range(k)]
    want = [s for (_, _, s) in sorted(slots)]
    assert list(d["perm"]) == want
    assert sorted(d["perm"]) == list(range(T * k))                       # bijection
    assert (d["inv"][d["perm"]] == np.arange(T * k)).all()
    assert d["counts"].sum() == T * k and d["seg_off"][0] == 0 and d["seg_off"][-1] == T * k
    np.testing.assert_array_equal(d["counts"], np.bincount(idx.reshape(-1), minlength=N))
    for e in range(N):
        seg = d["perm"][d["seg_off"][e]:d["seg_off"][e + 1]]
        assert (idx.reshape(-1)[seg] == e).all()
        assert (np.diff(seg // k) > 0).all()                             # token ascending


def test_dispatch_handles_empty_experts():
    idx = np.array([[2], [2], [0]], np.int32)
    d = orc.dispatch(idx, 4)
    assert list(d["counts"]) == [1, 0, 2, 0]
    assert list(d["seg_off"]) == [0, 1, 1, 3, 3]
    assert list(d["perm"]) == [2, 0, 1]


# ---- auxiliary loss (identity (c) and the worked example) -------------------
def test_aux_loss_worked_example():
    with open(os.path.join(HERE, "golden", "aux_loss_n2_t4.json")) as fh:
        g = json.load(fh)
    probs = np.array(g["probs"])
    idx = np.array(g["argmax"], np.int32)[:, None]
    loss, F, P = orc.aux_loss(probs, idx, g["coef"])
    np.testing.assert_allclose(F, g["F"], rtol=1e-15)
    np.testing.assert_allclose(P, g["P"], rtol=1e-15)
    assert loss == pytest.approx(g["loss"], rel=1e-14)


def test_aux_loss_worked_example_where_the_two_counting_modes_differ():
    # Eq. 9 counts the arg-max expert; the sentence under it speaks of the tokens dispatched to expert i, which
    # with top-2 is every selection.  Worked by hand for N = 3, T = 4: the two readings give different F and loss.
    with open(os.path.join(HERE, "golden", "aux_loss_n3_t4_k2.json")) as fh:
        g = json.load(fh)
    probs = np.array(g["probs"])
    idx = np.array(g["expert_idx"], np.int32)
    for mode in (0, 1):
        loss, F, P = orc.aux_loss(probs, idx, g["coef"], f_mode=mode)
        np.testing.assert_allclose(F, g[f"mode{mode}"]["F"], rtol=1e-15, atol=0)
        np.testing.assert_allclose(P, g["P"], rtol=1e-15)
        assert loss == pytest.approx(g[f"mode{mode}"]["loss"], rel=1e-14)
        count, psum = orc.aux_sums(probs, idx, f_mode=mode)
        assert list(count) == g[f"counts_mode{mode}"]
        np.testing.assert_allclose(psum, g["prob_sums"], rtol=1e-15)
    assert g["mode0"]["loss"] != g["mode1"]["loss"]


@pytest.mark.parametrize("mode", [0, 1])
def test_aux_sums_of_shards_add_up_to_the_loss_of_the_whole_batch(mode):
    # Eq. 8-9 are fractions of the whole batch: the loss is NOT the mean of the shards' losses, but the shards'
    # un-normalised sums add, and the loss from the added sums is the loss of the concatenated batch
    x, p, _, kw = make_case(T=37, N=5, seed=3)
    r = orc.router_forward(x, p["w_router"], None, 2)
    full, F, P = orc.aux_loss(r["probs"], r["expert_idx"], 0.3, f_mode=mode)
    cuts = [0, 9, 10, 30, 37]
    count = np.zeros(5)
    psum = np.zeros(5)
    shard_losses = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        c, s = orc.aux_sums(r["probs"][a:b], r["expert_idx"][a:b], f_mode=mode)
        count += c
        psum += s
        shard_losses.append(orc.aux_loss(r["probs"][a:b], r["expert_idx"][a:b], 0.3, f_mode=mode)[0])
    loss, F2, P2 = orc.aux_loss_from_sums(count, psum, 37, 2, 0.3, f_mode=mode)
    assert loss == pytest.approx(full, rel=1e-13)
    np.testing.assert_allclose(F2, F, rtol=1e-13)
    np.testing.assert_allclose(P2, P, rtol=1e-13)
    assert abs(np.mean(shard_losses) - full) > 1e-4          # the per-shard loss is a different quantity


@pytest.mark.parametrize("N", [2, 4, 8, 16])
def test_aux_loss_is_one_under_uniform_routing(N):
    # (i) F uniform through cyclic arg-max, P arbitrary-but-summing-to-one
    T = 4 * N
    logits = np.zeros((T, N))
    for t in range(T):
        logits[t, t % N] = 2.0
        logits[t, (t + 1) % N] = 1.0
    r = orc.router_forward(np.eye(T), logits.T.copy(), None, 2)
    loss, F, P = orc.aux_loss(r["probs"], r["expert_idx"], 1.0)
    np.testing.assert_allclose(F, 1.0 / N)
    assert loss == pytest.approx(1.0, rel=1e-13)
    # (ii) P uniform (all logits equal), F whatever the tie-break gives
    r = orc.router_forward(np.ones((T, 1)), np.ones((N, 1)), None, 2)
    loss, F, P = orc.aux_loss(r["probs"], r["expert_idx"], 1.0)
    np.testing.assert_allclose(P, 1.0 / N)
    assert F.sum() == pytest.approx(1.0) and loss == pytest.approx(1.0, rel=1e-13)
    # the second counting mode also sums to one
    loss, F, P = orc.aux_loss(r["probs"], r["expert_idx"], 1.0, f_mode=1)
    assert F.sum() == pytest.approx(1.0) and loss == pytest.approx(1.0, rel=1e-13)


def test_aux_loss_scales_with_coefficient_and_sums():
    x, p, _, kw = make_case(T=33, N=5)
    r = orc.router_forward(x, p["w_router"], None, 2)
    l1, F, P = orc.aux_loss(r["probs"], r["expert_idx"], 1.0)
    l2, _, _ = orc.aux_loss(r["probs"], r["expert_idx"], 0.01)
    assert l2 == pytest.approx(0.01 * l1)
    assert F.sum() == pytest.approx(1.0) and P.sum() == pytest.approx(1.0)


# ---- forward identities ----------------------------------------------------
def test_identity_a_zero_B_gives_the_frozen_ffn():
    x, p, _, kw = make_case(T=19, bias=True)
    for n in ("b_gate", "b_up", "b_down"):
        p[n] = np.zeros_like(p[n])
    y, _ = orc.ffn_forward(x, p, **kw)
    np.testing.assert_allclose(y, dense_ffn(x, p["w_gate"], p["w_up"], p["w_down"]), rtol=1e-12, atol=1e-13)


def test_identity_a_fails_without_renormalisation():
    # the identity needs the gates to sum to one: documents why Norm(.) is kept
    x, p, _, kw = make_case(T=19)
    for n in ("b_gate", "b_up", "b_down"):
        p[n] = np.zeros_like(p[n])
    y, _ = orc.ffn_forward(x, p, renormalize=False, **kw)
    ref = dense_ffn(x, p["w_gate"], p["w_up"], p["w_down"])
    assert np.abs(y - ref).max() > 1e-3 * np.abs(ref).max()


def test_identity_b_single_expert_is_plain_lora_on_the_ffn():
    x, p, _, kw = make_case(T=11, d=9, f=13, N=1, k=1, r=4, alpha=10.0)
    s = 10.0 / 4
    y, saved = orc.ffn_forward(x, p, **kw)
    np.testing.assert_allclose(saved["route"]["gates"], 1.0)
    ref = dense_ffn(x, p["w_gate"] + s * p["b_gate"][0] @ p["a_gate"][0],
                    p["w_up"] + s * p["b_up"][0] @ p["a_up"][0],
                    p["w_down"] + s * p["b_down"][0] @ p["a_down"][0])
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("k,N", [(1, 3), (2, 4), (3, 3)])
def test_shared_projection_form_equals_vanilla_form(k, N):
    x, p, _, kw = make_case(T=13, N=N, k=k, bias=True)
    y, _ = orc.ffn_forward(x, p, **kw)
    yv = orc.ffn_forward_vanilla(x, p, **kw)
    np.testing.assert_allclose(y, yv, rtol=1e-11, atol=1e-12)


def test_sparse_slices_equal_the_dense_masked_form():
    # Algorithm 1 keeps full shapes inside the expert loop: gate 0 for unselected experts
    x, p, _, kw = make_case(T=9, N=4, k=2)
    y, saved = orc.ffn_forward(x, p, **kw)
    s = kw["lora_alpha"] / p["a_gate"].shape[1]
    dense_gate = np.zeros((9, 4))
    np.put_along_axis(dense_gate, saved["route"]["expert_idx"].astype(np.int64), saved["route"]["gates"], axis=1)
    G, U = x @ p["w_gate"].T, x @ p["w_up"].T
    acc = np.zeros_like(y)
    for e in range(4):
        a = G + s * (x @ p["a_gate"][e].T) @ p["b_gate"][e].T
        b = U + s * (x @ p["a_up"][e].T) @ p["b_up"][e].T
        h = a * scipy.special.expit(a) * b
        acc += dense_gate[:, e:e + 1] * (h @ p["w_down"].T + s * (h @ p["a_down"][e].T) @ p["b_down"][e].T)
    np.testing.assert_allclose(y, acc, rtol=1e-11, atol=1e-12)


def test_token_forward_equals_the_batched_forward():
    x, p, _, kw = make_case(T=6, bias=True)
    y, _ = orc.ffn_forward(x, p, **kw)
    for t in range(6):
        yt, _ = orc.token_forward(x[t], p, **kw)
        np.testing.assert_allclose(yt, y[t], rtol=1e-11, atol=1e-12)


def test_forced_routing_changes_only_the_forced_tokens():
    x, p, _, kw = make_case(T=8, N=4, k=2)
    y, saved = orc.ffn_forward(x, p, **kw)
    idx = saved["route"]["expert_idx"].copy()
    idx[3] = idx[3][::-1]                      # same set, other order: same output
    y2, _ = orc.ffn_forward(x, p, forced_expert_idx=idx, **kw)
    np.testing.assert_allclose(y2, y, rtol=1e-12, atol=1e-13)
    others = [e for e in range(4) if e not in idx[5]]
    idx[5] = others[:2]
    y3, _ = orc.ffn_forward(x, p, forced_expert_idx=idx, **kw)
    keep = [t for t in range(8) if t != 5]
    np.testing.assert_allclose(y3[keep], y[keep], rtol=1e-12, atol=1e-13)
    assert np.abs(y3[5] - y[5]).max() > 1e-6


# ---- backward: identity (d), central differences ---------------------------
def total_loss(x, p, dy, kw, coef, f_mode=0, renormalize=True):
    y, saved = orc.ffn_forward(x, p, renormalize=renormalize, **kw)
    la, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], coef, f_mode)
    return float(np.sum(dy * y)) + la


@pytest.mark.parametrize("k,N,renorm,coef,f_mode", [(2, 3, True, 0.7, 0), (3, 3, True, 0.0, 0), (2, 4, False, 0.3, 0),
                                                    (1, 3, True, 0.5, 0), (2, 4, True, 0.9, 1), (2, 3, False, 0.4, 1)])
def test_identity_d_finite_differences(k, N, renorm, coef, f_mode):
    x, p, dy, kw = make_case(T=5, d=8, f=12, N=N, k=k, r=2, alpha=4.0, seed=11 + k, bias=True)
    # keep routing margins far above the step so the discrete choice is constant
    assert orc.router_forward(x, p["w_router"], p["router_bias"], k)["margin"].min() > 1e-3
    y, saved = orc.ffn_forward(x, p, renormalize=renorm, **kw)
    g = orc.ffn_backward(x, p, dy, saved, aux_coef=coef, aux_f_mode=f_mode)
    if f_mode == 1:
        # the case must tell the two counting modes apart: P is not uniform, the two F differ, and so do the
        # router gradients (a mode 1 that silently computed mode 0 would pass a comparison with itself)
        _, F0, P = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], coef, 0)
        _, F1, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], coef, 1)
        assert np.abs(P - 1.0 / N).max() > 0.02 and np.abs(F0 - F1).max() > 0.05
        g0 = orc.ffn_backward(x, p, dy, saved, aux_coef=coef, aux_f_mode=0)
        assert np.abs(g0["d_w_router"] - g["d_w_router"]).max() > 1e-4
    step = 1e-6
    rng = np.random.default_rng(5)

    def check(name, arr, grad):
        flat = arr.reshape(-1)
        picks = rng.choice(flat.size, size=min(flat.size, 25), replace=False)
        for i in picks:
            old = flat[i]
            flat[i] = old + step
            lp = total_loss(x, p, dy, kw, coef, f_mode=f_mode, renormalize=renorm)
            flat[i] = old - step
            lm = total_loss(x, p, dy, kw, coef, f_mode=f_mode, renormalize=renorm)
            flat[i] = old
            fd = (lp - lm) / (2 * step)
            assert grad.reshape(-1)[i] == pytest.approx(fd, rel=2e-5, abs=2e-7), (name, i)

    for name in ("a_gate", "b_gate", "a_up", "b_up", "a_down", "b_down"):
        check(name, p[name], g["d_" + name])
    check("w_router", p["w_router"], g["d_w_router"])
    check("router_bias", p["router_bias"], g["d_router_bias"])
    check("x", x, g["d_x"])


@pytest.mark.parametrize("mode", [0, 1])
def test_shard_gradients_with_the_batch_statistics_add_up_to_the_full_batch_gradient(mode):
    # data parallel over tokens: every term of the backward pass is a sum over tokens once the aux term uses the
    # whole batch's F_i and token count (Eq. 8-9), so the shards' gradients add up to the full-batch gradient
    x, p, dy, kw = make_case(T=12, d=8, f=10, N=4, k=2, r=2, seed=21, bias=True)
    coef = 0.8
    _, saved = orc.ffn_forward(x, p, **kw)
    full = orc.ffn_backward(x, p, dy, saved, aux_coef=coef, aux_f_mode=mode)
    cuts = [0, 5, 12]
    count = np.zeros(4)
    psum = np.zeros(4)
    shards = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        _, sv = orc.ffn_forward(x[a:b], p, **kw)
        c, s = orc.aux_sums(sv["route"]["probs"], sv["route"]["expert_idx"], f_mode=mode)
        count += c
        psum += s
        shards.append((a, b, sv))
    _, F, _ = orc.aux_loss_from_sums(count, psum, 12, 2, coef, f_mode=mode)
    total = None
    dx = np.zeros_like(x)
    for a, b, sv in shards:
        g = orc.ffn_backward(x[a:b], p, dy[a:b], sv, aux_coef=coef, aux_f_mode=mode, aux_batch=(F, 12))
        dx[a:b] = g["d_x"]
        part = {n: g[n] for n in g if n.startswith("d_") and n not in ("d_x", "d_gates", "d_logits")}
        total = part if total is None else {n: total[n] + part[n] for n in part}
    for n in total:
        np.testing.assert_allclose(total[n], full[n], rtol=1e-11, atol=1e-13, err_msg=n)
    np.testing.assert_allclose(dx, full["d_x"], rtol=1e-11, atol=1e-13)
    # with the shards' own statistics instead, the router gradient is a different one
    g_local = orc.ffn_backward(x[:5], p, dy[:5], shards[0][2], aux_coef=coef, aux_f_mode=mode)
    g_batch = orc.ffn_backward(x[:5], p, dy[:5], shards[0][2], aux_coef=coef, aux_f_mode=mode, aux_batch=(F, 12))
    assert np.abs(g_local["d_w_router"] - g_batch["d_w_router"]).max() > 1e-3


def test_backward_without_dx_leaves_other_gradients_unchanged():
    x, p, dy, kw = make_case()
    _, saved = orc.ffn_forward(x, p, **kw)
    g1 = orc.ffn_backward(x, p, dy, saved, aux_coef=0.1)
    g2 = orc.ffn_backward(x, p, dy, saved, aux_coef=0.1, want_dx=False)
    assert g2["d_x"] is None
    for n in g1:
        if n != "d_x":
            np.testing.assert_array_equal(g1[n], g2[n])


def test_frozen_ffn_gradient_when_B_is_zero_matches_dense_autodiff_by_differences():
    # with B = 0 the LoRA-A gradients vanish and dx equals that of the dense FFN plus the router path
    x, p, dy, kw = make_case(T=4, d=6, f=8, N=3, k=2, r=2)
    for n in ("b_gate", "b_up", "b_down"):
        p[n] = np.zeros_like(p[n])
    _, saved = orc.ffn_forward(x, p, **kw)
    g = orc.ffn_backward(x, p, dy, saved)
    for n in ("d_a_gate", "d_a_up", "d_a_down"):
        assert np.abs(g[n]).max() == 0.0
    # gates sum to one and every expert output is identical => the router gets no gradient
    assert np.abs(g["d_w_router"]).max() < 1e-12
    step = 1e-6
    fd = np.zeros_like(x)
    for i in range(x.size):
        xp = x.copy().reshape(-1); xp[i] += step
        xm = x.copy().reshape(-1); xm[i] -= step
        fp = np.sum(dy * dense_ffn(xp.reshape(x.shape), p["w_gate"], p["w_up"], p["w_down"]))
        fm = np.sum(dy * dense_ffn(xm.reshape(x.shape), p["w_gate"], p["w_up"], p["w_down"]))
        fd.reshape(-1)[i] = (fp - fm) / (2 * step)
    np.testing.assert_allclose(g["d_x"], fd, rtol=1e-5, atol=1e-7)


# ---- planted mistakes: the pins above must notice them ----------------------
def test_pins_catch_a_wrong_lora_scale(monkeypatch):
    x, p, _, kw = make_case(T=11, d=9, f=13, N=1, k=1, r=4, alpha=10.0)
    y, _ = orc.ffn_forward(x, p, top_k=1, lora_alpha=4.0)        # as if s were 1 instead of alpha / r
    s = 10.0 / 4
    ref = dense_ffn(x, p["w_gate"] + s * p["b_gate"][0] @ p["a_gate"][0],
                    p["w_up"] + s * p["b_up"][0] @ p["a_up"][0],
                    p["w_down"] + s * p["b_down"][0] @ p["a_down"][0])
    assert np.abs(y - ref).max() > 1e-3


def test_pins_catch_a_wrong_silu_derivative(monkeypatch):
    x, p, dy, kw = make_case(T=5, d=8, f=12, N=3, k=2, r=2, alpha=4.0, seed=13)
    monkeypatch.setattr(orc, "silu_grad", lambda v: 1.0 / (1.0 + np.exp(-v)))    # drops a term
    _, saved = orc.ffn_forward(x, p, **kw)
    g = orc.ffn_backward(x, p, dy, saved)
    step = 1e-6
    arr = p["a_gate"].reshape(-1)
    worst = 0.0
    for i in range(0, arr.size, 7):
        old = arr[i]
        arr[i] = old + step; lp = total_loss(x, p, dy, kw, 0.0)
        arr[i] = old - step; lm = total_loss(x, p, dy, kw, 0.0)
        arr[i] = old
        worst = max(worst, abs((lp - lm) / (2 * step) - g["d_a_gate"].reshape(-1)[i]))
    assert worst > 1e-4


# ---- the block inside its layer (Eq. 5 / Eq. 6) -------------------------------
def test_rmsnorm_rows_have_unit_mean_square_and_ignore_the_input_scale():
    rng = np.random.default_rng(3)
    z = rng.normal(size=(6, 16)) * 3.0
    xn, inv = orc.rmsnorm(z, np.ones(16), 0.0)
    np.testing.assert_allclose(np.mean(xn * xn, axis=1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(inv, 1.0 / np.linalg.norm(z, axis=1) * np.sqrt(16), rtol=1e-12)
    xn2, _ = orc.rmsnorm(7.5 * z, np.ones(16), 0.0)
    np.testing.assert_allclose(xn2, xn, rtol=1e-12)
    # the weight is per channel, and eps enters under the root
    w = rng.normal(size=16)
    xn3, _ = orc.rmsnorm(z, w, 0.0)
    np.testing.assert_allclose(xn3, xn * w[None, :], rtol=1e-12)
    one = np.full((1, 4), 2.0)
    np.testing.assert_allclose(orc.rmsnorm(one, np.ones(4), 5.0)[0], 2.0 / 3.0, rtol=1e-12)   # 2 / sqrt(4 + 5)


def test_layer_is_the_residual_stream_plus_the_block_on_the_normalised_input():
    z, p, dh, kw = make_case(T=6, d=8, f=12, N=3, k=2, r=2)
    w = np.linspace(0.5, 1.5, 8)
    h, saved = orc.layer_forward(z, p, w, 1e-5, **kw)
    xn = z / np.sqrt(np.mean(z * z, axis=1, keepdims=True) + 1e-5) * w
    y, _ = orc.ffn_forward(xn, p, **kw)
    np.testing.assert_allclose(h, z + y, rtol=1e-12, atol=1e-12)
    # a block whose down projections are zero leaves the residual stream untouched, and its input gradient is dh
    p0 = dict(p, w_down=np.zeros_like(p["w_down"]), b_down=np.zeros_like(p["b_down"]))
    h0, s0 = orc.layer_forward(z, p0, w, 1e-5, **kw)
    np.testing.assert_array_equal(h0, z)
    g0 = orc.layer_backward(z, p0, w, dh, s0, aux_coef=0.0)
    np.testing.assert_allclose(g0["d_x"], dh, rtol=0, atol=1e-14)


def layer_loss(z, p, w, eps, dh, kw, coef):
    h, saved = orc.layer_forward(z, p, w, eps, **kw)
    la, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], coef)
    return float(np.sum(dh * h)) + la


@pytest.mark.parametrize("k,N,coef", [(2, 3, 0.6), (1, 4, 0.0)])
def test_layer_backward_matches_central_differences(k, N, coef):
    z, p, dh, kw = make_case(T=5, d=8, f=12, N=N, k=k, r=2, alpha=4.0, seed=21 + k, bias=True)
    z = z * 1.7
    w = np.random.default_rng(8).normal(size=8) * 0.3 + 1.0
    eps = 1e-3
    h, saved = orc.layer_forward(z, p, w, eps, **kw)
    assert saved["route"]["margin"].min() > 1e-3
    g = orc.layer_backward(z, p, w, dh, saved, aux_coef=coef)
    step = 1e-6

    def check(arr, grad, count, name):
        flat = arr.reshape(-1)
        for i in np.random.default_rng(2).choice(flat.size, size=min(flat.size, count), replace=False):
            old = flat[i]
            flat[i] = old + step
            lp = layer_loss(z, p, w, eps, dh, kw, coef)
            flat[i] = old - step
            lm = layer_loss(z, p, w, eps, dh, kw, coef)
            flat[i] = old
            assert grad.reshape(-1)[i] == pytest.approx((lp - lm) / (2 * step), rel=2e-5, abs=2e-7), (name, i)

    check(z, g["d_x"], 40, "z")
    check(p["a_gate"], g["d_a_gate"], 10, "a_gate")
    check(p["b_down"], g["d_b_down"], 10, "b_down")
    check(p["w_router"], g["d_w_router"], 10, "w_router")


def test_layer_pins_catch_a_dropped_projection_term_in_the_norm_gradient(monkeypatch):
    # without the `xh * mean(u * xh)` term the gradient is not orthogonal to z (for eps = 0 the normalised
    # vector does not change along z, so <dL/dz - dh, z> must vanish)
    z, p, dh, kw = make_case(T=5, d=8, f=12, N=3, k=2, r=2, seed=4)
    w = np.ones(8)
    h, saved = orc.layer_forward(z, p, w, 0.0, **kw)
    g = orc.layer_backward(z, p, w, dh, saved)
    np.testing.assert_allclose(np.sum((g["d_x"] - dh) * z, axis=1), 0.0, atol=1e-10)


# ---- plain LoRA linear (Eq. 1) -------------------------------------------------
def test_lora_linear_equals_the_merged_weight_of_eq_1():
    rng = np.random.default_rng(12)
    x, w = rng.normal(size=(9, 6)), rng.normal(size=(5, 6))
    a, b = rng.normal(size=(3, 6)), rng.normal(size=(5, 3))
    y = orc.lora_linear_forward(x, w, a, b, 6.0)
    np.testing.assert_allclose(y, x @ (w + (6.0 / 3) * b @ a).T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.lora_linear_forward(x, w, a, np.zeros_like(b), 6.0), x @ w.T, rtol=1e-13)


def test_lora_linear_backward_matches_central_differences():
    rng = np.random.default_rng(13)
    x, w = rng.normal(size=(7, 5)), rng.normal(size=(4, 5))
    a, b = rng.normal(size=(2, 5)), rng.normal(size=(4, 2))
    dy = rng.normal(size=(7, 4))
    g = orc.lora_linear_backward(x, w, a, b, 3.0, dy)
    step = 1e-6
    for name, arr in (("d_x", x), ("d_a", a), ("d_b", b)):
        flat = arr.reshape(-1)
        for i in range(flat.size):
            old = flat[i]
            flat[i] = old + step
            lp = np.sum(dy * orc.lora_linear_forward(x, w, a, b, 3.0))
            flat[i] = old - step
            lm = np.sum(dy * orc.lora_linear_forward(x, w, a, b, 3.0))
            flat[i] = old
            assert g[name].reshape(-1)[i] == pytest.approx((lp - lm) / (2 * step), rel=1e-6, abs=1e-8), (name, i)

