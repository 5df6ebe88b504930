"""CPU oracle for MixDoRA: the MixLoRA feed-forward block with every expert's LoRA replaced by DoRA
(arXiv 2404.15159, Section 4.1 and Table 1 name the variant; the paper prints no formula for it).

TEST INFRASTRUCTURE ONLY, like `mixlora_oracle`: float64 numpy, plain and slow, shares no code with the
CUDA path and is never called from a product code path.

Reading taken here (the paper is silent; this is the weight-decomposed adaptation of Liu et al. 2024 as the
common open implementations apply it to a linear layer with weight W [out, in]):

    W'_e = diag(m_e / n_e) (W + s B_e A_e),     n_e[o] = || W[o, :] + s B_e[o, :] A_e ||_2

  * one trainable magnitude per OUTPUT feature and expert: m_gate, m_up [N, f], m_down [N, d];
  * the norm n_e runs over the input dimension of each output row of the merged weight;
  * n_e is treated as a constant in the backward pass (no gradient flows through the norm), so the
    gradients are those of  y = c (W x + s B A x)  with the vector c = m / n held fixed for A and B,
    and  d m[o] = sum over the expert's slots of  dL/dout[o] * (W x + s B A x)[o] / n[o];
  * with m = n the block is exactly MixLoRA; with B = 0 and m = the row norms of W it is the frozen FFN;
  * the router, the top-k gates, the dispatch and the auxiliary loss are those of MixLoRA.

Each expert of the block is then (Algorithm 1's expert loop with the three scaled projections)

    a = c_g,e * (W1 x + s B_g,e A_g,e x),  b = c_u,e * (W3 x + s B_u,e A_u,e x),  h = SiLU(a) * b,
    o = c_d,e * (W2 h + s B_d,e A_d,e h),  y = sum_j g_j o_j.

The shared W1 x, W3 x of Section 3.3 (I) survive (the scale acts on the output rows); the frozen W2 can no
longer be applied once to the gate-weighted sum of a token's slots, because c_d differs between experts.
"""
from __future__ import annotations

import numpy as np

from . import mixlora_oracle as base

F64 = np.float64


def row_norms(w, a, b, s):
    """n[e, o] = || w[o, :] + s * b[e, o, :] @ a[e] ||_2 from the merged weight itself.  w [out, in],
    a [N, r, in], b [N, out, r]."""
    w, a, b = (np.asarray(v, F64) for v in (w, a, b))
    out = np.empty((a.shape[0], w.shape[0]), F64)
    for e in range(a.shape[0]):
        merged = w + s * (b[e] @ a[e])
        out[e] = np.sqrt(np.sum(merged * merged, axis=1))
    return out


def all_norms(params, lora_alpha):
    """The three norm tables of the block: dict(gate [N, f], up [N, f], down [N, d])."""
    r = np.asarray(params["a_gate"]).shape[1]
    s = float(lora_alpha) / r
    return dict(gate=row_norms(params["w_gate"], params["a_gate"], params["b_gate"], s),
                up=row_norms(params["w_up"], params["a_up"], params["b_up"], s),
                down=row_norms(params["w_down"], params["a_down"], params["b_down"], s))


def ffn_forward(x, params, magn, top_k, lora_alpha, renormalize=True, forced_expert_idx=None, norms=None):
    """MixDoRA block forward.  `magn` = dict(gate, up, down) of magnitudes; `norms` (optional, same keys)
    replaces the norms of the current merged weights (used to hold them fixed while A, B are perturbed, which
    is what 'no gradient through the norm' means).  Returns (y [T, d], saved)."""
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    M = {n: np.asarray(v, F64) for n, v in magn.items()}
    x = np.asarray(x, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s = float(lora_alpha) / r
    nrm = all_norms(P, lora_alpha) if norms is None else {n: np.asarray(v, F64) for n, v in norms.items()}
    c = {n: M[n] / nrm[n] for n in ("gate", "up", "down")}

    route = base.router_forward(x, P["w_router"], P.get("router_bias"), top_k, renormalize)
    if forced_expert_idx is not None:
        idx = np.asarray(forced_expert_idx, np.int32)
        sel = np.take_along_axis(route["probs"], idx.astype(np.int64), axis=1)
        route["expert_idx"] = idx
        route["gates"] = sel / sel.sum(axis=1, keepdims=True) if renormalize else sel
    disp = base.dispatch(route["expert_idx"], N)

    G = x @ P["w_gate"].T                               # shared by all experts, once per token
    U = x @ P["w_up"].T
    y = np.zeros((T, d), F64)
    gates_flat = route["gates"].reshape(-1)
    per_expert = []
    for e in range(N):
        slots = disp["perm"][disp["seg_off"][e]:disp["seg_off"][e + 1]].astype(np.int64)
        tok = slots // top_k
        xe = x[tok]
        zg = xe @ P["a_gate"][e].T
        zu = xe @ P["a_up"][e].T
        a_pre = G[tok] + s * (zg @ P["b_gate"][e].T)
        b_pre = U[tok] + s * (zu @ P["b_up"][e].T)
        a = c["gate"][e][None, :] * a_pre
        b = c["up"][e][None, :] * b_pre
        h = base.silu(a) * b
        zd = h @ P["a_down"][e].T
        o_pre = h @ P["w_down"].T + s * (zd @ P["b_down"][e].T)
        o = c["down"][e][None, :] * o_pre
        g = gates_flat[slots]
        y[tok] += g[:, None] * o
        per_expert.append(dict(slots=slots, tok=tok, zg=zg, zu=zu, a_pre=a_pre, b_pre=b_pre, a=a, b=b, h=h, zd=zd,
                               o_pre=o_pre, o=o, g=g))
    saved = dict(route=route, disp=disp, per_expert=per_expert, s=s, top_k=top_k, renormalize=renormalize,
                 norms=nrm, scales=c)
    return y, saved


def ffn_forward_merged(x, params, magn, top_k, lora_alpha, renormalize=True):
    """Plain definition: every selected expert is a whole FFN with the three DoRA weights W'_e formed
    explicitly, applied token by token."""
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x = np.asarray(x, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s = float(lora_alpha) / r
    route = base.router_forward(x, P["w_router"], P.get("router_bias"), top_k, renormalize)

    def dora(w, a, b, m):
        merged = w + s * (b @ a)
        return (np.asarray(m, F64) / np.sqrt(np.sum(merged * merged, axis=1)))[:, None] * merged

    y = np.zeros((T, d), F64)
    for t in range(T):
        for j in range(top_k):
            e = int(route["expert_idx"][t, j])
            w1 = dora(P["w_gate"], P["a_gate"][e], P["b_gate"][e], magn["gate"][e])
            w3 = dora(P["w_up"], P["a_up"][e], P["b_up"][e], magn["up"][e])
            w2 = dora(P["w_down"], P["a_down"][e], P["b_down"][e], magn["down"][e])
            h = base.silu(w1 @ x[t]) * (w3 @ x[t])
            y[t] += route["gates"][t, j] * (w2 @ h)
    return y


def ffn_backward(x, params, magn, dy, saved, aux_coef=0.0, aux_f_mode=0, want_dx=True):
    """Gradients of L = sum(dy * y) + L_aux with the norms held constant: LoRA matrices, magnitudes
    (d_m_gate, d_m_up [N, f], d_m_down [N, d]), router, and optionally x."""
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x = np.asarray(x, F64)
    dy = np.asarray(dy, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s, k, route = saved["s"], saved["top_k"], saved["route"]
    c, nrm = saved["scales"], saved["norms"]

    g_ag = np.zeros_like(P["a_gate"]); g_bg = np.zeros_like(P["b_gate"])
    g_au = np.zeros_like(P["a_up"]);   g_bu = np.zeros_like(P["b_up"])
    g_ad = np.zeros_like(P["a_down"]); g_bd = np.zeros_like(P["b_down"])
    g_mg = np.zeros_like(nrm["gate"]); g_mu = np.zeros_like(nrm["up"]); g_md = np.zeros_like(nrm["down"])
    dx = np.zeros((T, d), F64)
    dgate = np.zeros(T * k, F64)

    for e in range(N):
        E = saved["per_expert"][e]
        tok, slots = E["tok"], E["slots"]
        dye = dy[tok]
        dgate[slots] = np.sum(dye * E["o"], axis=1)
        do = E["g"][:, None] * dye                               # dL/do (scaled output)
        g_md[e] = np.sum(do * E["o_pre"], axis=0) / nrm["down"][e]
        do_pre = do * c["down"][e][None, :]
        g_bd[e] = s * (do_pre.T @ E["zd"])
        dzd = s * (do_pre @ P["b_down"][e])
        g_ad[e] = dzd.T @ E["h"]
        dh = do_pre @ P["w_down"] + dzd @ P["a_down"][e]
        da = dh * E["b"] * base.silu_grad(E["a"])                # dL/da, dL/db (scaled pre-activations)
        db = dh * base.silu(E["a"])
        g_mg[e] = np.sum(da * E["a_pre"], axis=0) / nrm["gate"][e]
        g_mu[e] = np.sum(db * E["b_pre"], axis=0) / nrm["up"][e]
        da_pre = da * c["gate"][e][None, :]
        db_pre = db * c["up"][e][None, :]
        xe = x[tok]
        g_bg[e] = s * (da_pre.T @ E["zg"])
        dzg = s * (da_pre @ P["b_gate"][e])
        g_ag[e] = dzg.T @ xe
        g_bu[e] = s * (db_pre.T @ E["zu"])
        dzu = s * (db_pre @ P["b_up"][e])
        g_au[e] = dzu.T @ xe
        if want_dx:
            dx[tok] += (da_pre @ P["w_gate"] + db_pre @ P["w_up"] + dzg @ P["a_gate"][e] + dzu @ P["a_up"][e])

    dgate = dgate.reshape(T, k)
    probs = route["probs"]
    idx = route["expert_idx"].astype(np.int64)
    dp = np.zeros((T, N), F64)
    if saved["renormalize"]:
        q = np.take_along_axis(probs, idx, axis=1).sum(axis=1, keepdims=True)
        inner = np.sum(route["gates"] * dgate, axis=1, keepdims=True)
        np.put_along_axis(dp, idx, (dgate - inner) / q, axis=1)
    else:
        np.put_along_axis(dp, idx, dgate, axis=1)
    if aux_coef != 0.0:
        _, F, _ = base.aux_loss(probs, route["expert_idx"], aux_coef, aux_f_mode)
        dp += (aux_coef * N / T) * F[None, :]
    dl = probs * (dp - np.sum(probs * dp, axis=1, keepdims=True))
    g_wr = dl.T @ x
    g_br = dl.sum(axis=0)
    if want_dx:
        dx += dl @ P["w_router"]
    return dict(d_a_gate=g_ag, d_b_gate=g_bg, d_a_up=g_au, d_b_up=g_bu, d_a_down=g_ad, d_b_down=g_bd,
                d_m_gate=g_mg, d_m_up=g_mu, d_m_down=g_md, d_w_router=g_wr, d_router_bias=g_br,
                d_x=dx if want_dx else None, d_gates=dgate, d_logits=dl)
