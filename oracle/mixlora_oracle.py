"""CPU oracle for the MixLoRA feed-forward block (arXiv 2404.15159).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the CUDA
library is checked against.  It shares no code with the CUDA path, imports
nothing from the package, and must never be called from a product code path:
only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

Everything is float64 numpy.  Dense products (`@`) are the only library
primitive; there is no tiling, fusion or reordering beyond what the paper states.

Notation (paper): T tokens, d = model width, f = FFN width, N experts, k = top-k,
r = LoRA rank, s = alpha / r.  W1 = gate, W3 = up, W2 = down (Section 3.3).
Weights are stored [out, in] as in Eq. 1 (W in R^{d1 x d2}, W' = W + B A):

    w_gate, w_up : [f, d]      w_down : [d, f]      w_router : [N, d]
    a_gate, a_up : [N, r, d]   b_gate, b_up : [N, f, r]
    a_down       : [N, r, f]   b_down       : [N, d, r]

A *slot* is one (token, selected expert) pair; slot id = t * k + j where j is the
rank of the expert among the token's k choices (j = 0 is the largest logit).

Readings of the paper where it is silent or inconsistent:
  * gates are re-normalised over the k selected experts (Algorithm 1 applies
    Norm(Top2(Softmax(.))); Eq. 7 omits the Norm);
  * selection is on the logits (monotone in the softmax), ties go to the lower
    expert index;
  * F_i of Eq. 9 counts the arg-max expert only (f_mode 1: every selection, the
    reading of the sentence under Eq. 9; both are pinned by a hand-worked
    example in which they differ); P_i is the mean of the full softmax
    probability.  PARITY UNPINNED for the choice of P_i (full softmax versus
    re-normalised gate): no identity in the paper tells them apart.
  * F_i and P_i are fractions of the whole batch: when the batch is split over
    data-parallel shards, the shards' sums are added before Eq. 8 is evaluated
    (`aux_sums`, `aux_loss_from_sums`, `aux_batch=` of the backward pass).
  * the LoRA scale is s = alpha / r (Table 3 lists alpha; Eq. 1 has no scale).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- #
# small pieces
# --------------------------------------------------------------------------- #
def softmax_rows(logits: np.ndarray) -> np.ndarray:
    """Softmax over the expert axis (Eq. 7)."""
    z = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=1, keepdims=True)


def silu(v: np.ndarray) -> np.ndarray:
    """SiLU(v) = v / (1 + exp(-v)) (Section 3.3, FFN of LLaMA)."""
    return v / (1.0 + np.exp(-v))


def silu_grad(v: np.ndarray) -> np.ndarray:
    """d SiLU / dv = sigma(v) * (1 + v * (1 - sigma(v)))."""
    sig = 1.0 / (1.0 + np.exp(-v))
    return sig * (1.0 + v * (1.0 - sig))


# --------------------------------------------------------------------------- #
# router (Eq. 7, Algorithm 1 steps "Linear" and "Norm(Top2(Softmax))")
# --------------------------------------------------------------------------- #
def router_forward(x, w_router, router_bias, top_k, renormalize=True):
    """Top-k softmax router.

    Returns a dict with
      logits [T,N], probs [T,N], expert_idx [T,k] (descending logit, ties to the
      lower index), gates [T,k], margin [T] (smallest logit gap that decides a
      discrete choice: l_(k) - l_(k+1) and, for the arg-max of Eq. 9,
      l_(1) - l_(2); +inf where no such gap exists).
    """
    x = np.asarray(x, F64)
    w_router = np.asarray(w_router, F64)
    T = x.shape[0]
    N = w_router.shape[0]
    logits = x @ w_router.T
    if router_bias is not None:
        logits = logits + np.asarray(router_bias, F64)[None, :]
    probs = softmax_rows(logits)
    order = np.argsort(-logits, axis=1, kind="stable")  # stable: ties -> lower index
    expert_idx = order[:, :top_k].astype(np.int32)
    sel = np.take_along_axis(probs, expert_idx.astype(np.int64), axis=1)
    if renormalize:
        gates = sel / sel.sum(axis=1, keepdims=True)
    else:
        gates = sel
    sorted_l = np.take_along_axis(logits, order, axis=1)
    margin = np.full(T, np.inf)
    if top_k < N:
        margin = np.minimum(margin, sorted_l[:, top_k - 1] - sorted_l[:, top_k])
    if N > 1:
        margin = np.minimum(margin, sorted_l[:, 0] - sorted_l[:, 1])
    return dict(logits=logits, probs=probs, expert_idx=expert_idx, gates=gates, margin=margin)


# --------------------------------------------------------------------------- #
# dispatch: histogram, prefix scan, stable permutation
# --------------------------------------------------------------------------- #
def dispatch(expert_idx: np.ndarray, n_experts: int):
    """Group the T*k slots by expert (Section 3.3: each expert works on its slice).

    Canonical order: expert ascending, then token ascending (a token's k experts
    are distinct, so the key is unique).  Returns
      counts [N], seg_off [N+1] (exclusive scan), perm [T*k] (slot id at each
      sorted position), inv [T*k] (sorted position of each slot id).
    """
    T, k = expert_idx.shape
    counts = np.zeros(n_experts, np.int64)
    for e in expert_idx.reshape(-1):
        counts[e] += 1
    seg_off = np.zeros(n_experts + 1, np.int64)
    seg_off[1:] = np.cumsum(counts)
    cursor = seg_off[:-1].copy()
    perm = np.empty(T * k, np.int64)
    inv = np.empty(T * k, np.int64)
    for t in range(T):            # token ascending => stable inside each expert
        for j in range(k):
            e = expert_idx[t, j]
            pos = cursor[e]
            cursor[e] += 1
            perm[pos] = t * k + j
            inv[t * k + j] = pos
    return dict(counts=counts.astype(np.int32), seg_off=seg_off.astype(np.int32),
                perm=perm.astype(np.int32), inv=inv.astype(np.int32))


# --------------------------------------------------------------------------- #
# auxiliary load-balance loss (Eq. 8-9)
# --------------------------------------------------------------------------- #
def aux_loss(probs, expert_idx, coef, f_mode=0):
    """L_aux = coef * N * sum_i F_i * P_i.

    f_mode 0: F_i = share of tokens whose arg-max expert is i (Eq. 9 as printed).
    f_mode 1: F_i = share of the T*k selections that went to expert i.
    P_i = mean over tokens of the softmax probability of expert i.
    """
    T, N = probs.shape
    k = expert_idx.shape[1]
    F = np.zeros(N, F64)
    if f_mode == 0:
        for t in range(T):
            F[expert_idx[t, 0]] += 1.0
        F /= T
    else:
        for e in expert_idx.reshape(-1):
            F[e] += 1.0
        F /= T * k
    P = probs.sum(axis=0) / T
    loss = coef * N * float(np.dot(F, P))
    return loss, F, P


def aux_sums(probs, expert_idx, f_mode=0):
    """The two sums over tokens that Eq. 9 is built from, un-normalised, for one batch or one shard of it:
    count[i] = tokens whose arg-max expert is i (f_mode 1: selections that went to i), prob_sum[i] = sum over
    tokens of the softmax probability of expert i.  Sums of shards add up to the sums of the whole batch."""
    T, N = probs.shape
    count = np.zeros(N, F64)
    if f_mode == 0:
        for t in range(T):
            count[expert_idx[t, 0]] += 1.0
    else:
        for e in expert_idx.reshape(-1):
            count[e] += 1.0
    return count, probs.sum(axis=0)


def aux_loss_from_sums(count, prob_sum, total_tokens, top_k, coef, f_mode=0):
    """Eq. 8-9 from the sums of `aux_sums` taken over ALL `total_tokens` tokens of the batch (F_i and P_i are
    fractions of the whole batch, so under data parallelism the shard sums are added first)."""
    N = len(count)
    F = np.asarray(count, F64) / (total_tokens * (top_k if f_mode == 1 else 1))
    P = np.asarray(prob_sum, F64) / total_tokens
    return coef * N * float(np.dot(F, P)), F, P


# --------------------------------------------------------------------------- #
# forward, optimised form (Algorithm 1: shared W1/W3 results, per-expert slices)
# --------------------------------------------------------------------------- #
def ffn_forward(x, params, top_k, lora_alpha, renormalize=True, forced_expert_idx=None):
    """MixLoRA block forward (Eq. 6 read through Algorithm 1).

    `params` is a dict of the arrays listed in the module header (router_bias
    optional).  `forced_expert_idx` replaces the router's discrete choice (used
    to compare on identical routing when a margin is below the flag threshold);
    the gates are then taken from the softmax at the forced experts.

    Returns (y [T,d], saved) where `saved` holds routing, dispatch and the
    intermediates the backward pass needs.
    """
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x = np.asarray(x, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s = float(lora_alpha) / r

    route = router_forward(x, P["w_router"], P.get("router_bias"), top_k, renormalize)
    if forced_expert_idx is not None:
        idx = np.asarray(forced_expert_idx, np.int32)
        sel = np.take_along_axis(route["probs"], idx.astype(np.int64), axis=1)
        route["expert_idx"] = idx
        route["gates"] = sel / sel.sum(axis=1, keepdims=True) if renormalize else sel
    disp = dispatch(route["expert_idx"], N)

    # shared frozen projections, once per token (Section 3.3 (I))
    G = x @ P["w_gate"].T
    U = x @ P["w_up"].T

    y = np.zeros((T, d), F64)
    gates_flat = route["gates"].reshape(-1)
    per_expert = []
    for e in range(N):
        slots = disp["perm"][disp["seg_off"][e]:disp["seg_off"][e + 1]].astype(np.int64)
        tok = slots // top_k
        xe = x[tok]
        zg = xe @ P["a_gate"][e].T                      # [n_e, r]
        zu = xe @ P["a_up"][e].T
        a = G[tok] + s * (zg @ P["b_gate"][e].T)        # gate pre-activation
        b = U[tok] + s * (zu @ P["b_up"][e].T)          # up pre-activation
        h = silu(a) * b
        zd = h @ P["a_down"][e].T
        o = h @ P["w_down"].T + s * (zd @ P["b_down"][e].T)
        g = gates_flat[slots]
        y[tok] += g[:, None] * o                        # tokens are distinct inside a segment
        per_expert.append(dict(slots=slots, tok=tok, zg=zg, zu=zu, a=a, b=b, h=h, zd=zd, o=o, g=g))

    saved = dict(route=route, disp=disp, per_expert=per_expert, G=G, U=U, s=s, top_k=top_k,
                 renormalize=renormalize)
    return y, saved


# --------------------------------------------------------------------------- #
# forward, plain definition (Fig. 3(a)): every selected expert is a whole FFN
# with merged weights W + s * B A (Eq. 1), applied token by token
# --------------------------------------------------------------------------- #
def ffn_forward_vanilla(x, params, top_k, lora_alpha, renormalize=True):
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x = np.asarray(x, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s = float(lora_alpha) / r
    route = router_forward(x, P["w_router"], P.get("router_bias"), top_k, renormalize)
    merged = []
    for e in range(N):
        merged.append((P["w_gate"] + s * P["b_gate"][e] @ P["a_gate"][e],
                       P["w_up"] + s * P["b_up"][e] @ P["a_up"][e],
                       P["w_down"] + s * P["b_down"][e] @ P["a_down"][e]))
    y = np.zeros((T, d), F64)
    for t in range(T):
        for j in range(top_k):
            e = int(route["expert_idx"][t, j])
            w1, w3, w2 = merged[e]
            h = silu(w1 @ x[t]) * (w3 @ x[t])
            y[t] += route["gates"][t, j] * (w2 @ h)
    return y


# --------------------------------------------------------------------------- #
# backward (chain rule on the forward above; the paper prints none)
# --------------------------------------------------------------------------- #
def ffn_backward(x, params, dy, saved, aux_coef=0.0, aux_f_mode=0, want_dx=True, aux_batch=None):
    """Gradients of L = sum(dy * y) + L_aux with respect to the LoRA matrices,
    the router and (optionally) x.  The frozen weights get no gradient.

    `aux_batch` = (F [N], total_tokens): when x is one shard of a larger batch, L_aux of Eq. 8 is the loss of
    the whole batch, so its gradient uses the batch's F_i and token count instead of the shard's.

    Returns a dict: d_a_gate, d_b_gate, d_a_up, d_b_up, d_a_down, d_b_down,
    d_w_router, d_router_bias, d_x (or None), d_gates [T,k], d_logits [T,N].
    """
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x = np.asarray(x, F64)
    dy = np.asarray(dy, F64)
    T, d = x.shape
    N, r, _ = P["a_gate"].shape
    s = saved["s"]
    k = saved["top_k"]
    route = saved["route"]

    g_ag = np.zeros_like(P["a_gate"]); g_bg = np.zeros_like(P["b_gate"])
    g_au = np.zeros_like(P["a_up"]);   g_bu = np.zeros_like(P["b_up"])
    g_ad = np.zeros_like(P["a_down"]); g_bd = np.zeros_like(P["b_down"])
    dx = np.zeros((T, d), F64)
    dgate = np.zeros(T * k, F64)

    for e in range(N):
        E = saved["per_expert"][e]
        tok, slots = E["tok"], E["slots"]
        dye = dy[tok]
        dgate[slots] = np.sum(dye * E["o"], axis=1)          # y = sum_j g_j o_j
        do = E["g"][:, None] * dye
        g_bd[e] = s * (do.T @ E["zd"])                        # o = W2 h + s B (A h)
        dzd = s * (do @ P["b_down"][e])
        g_ad[e] = dzd.T @ E["h"]
        dh = do @ P["w_down"] + dzd @ P["a_down"][e]
        da = dh * E["b"] * silu_grad(E["a"])                  # h = SiLU(a) * b
        db = dh * silu(E["a"])
        xe = x[tok]
        g_bg[e] = s * (da.T @ E["zg"])
        dzg = s * (da @ P["b_gate"][e])
        g_ag[e] = dzg.T @ xe
        g_bu[e] = s * (db.T @ E["zu"])
        dzu = s * (db @ P["b_up"][e])
        g_au[e] = dzu.T @ xe
        if want_dx:
            dx[tok] += (da @ P["w_gate"] + db @ P["w_up"]
                        + dzg @ P["a_gate"][e] + dzu @ P["a_up"][e])

    # router: gates -> probabilities -> logits
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
        if aux_batch is None:
            _, F, _ = aux_loss(probs, route["expert_idx"], aux_coef, aux_f_mode)
            T_all = T
        else:
            F, T_all = np.asarray(aux_batch[0], F64), aux_batch[1]
        dp += (aux_coef * N / T_all) * F[None, :]             # F_i is piecewise constant; P_i = sum_t p_ti / T_all
    dl = probs * (dp - np.sum(probs * dp, axis=1, keepdims=True))
    g_wr = dl.T @ x
    g_br = dl.sum(axis=0)
    if want_dx:
        dx += dl @ P["w_router"]

    return dict(d_a_gate=g_ag, d_b_gate=g_bg, d_a_up=g_au, d_b_up=g_bu,
                d_a_down=g_ad, d_b_down=g_bd, d_w_router=g_wr, d_router_bias=g_br,
                d_x=dx if want_dx else None, d_gates=dgate, d_logits=dl)


# --------------------------------------------------------------------------- #
# one-token evaluation, for sampled checks at sizes where a full pass is slow
# --------------------------------------------------------------------------- #
def token_forward(x_t, params, top_k, lora_alpha, renormalize=True, forced_experts=None):
    """y_t for a single token, straight from Eq. 6 / Algorithm 1 (matrix-vector only)."""
    P = {n: (None if v is None else np.asarray(v, F64)) for n, v in params.items()}
    x_t = np.asarray(x_t, F64)
    r = P["a_gate"].shape[1]
    s = float(lora_alpha) / r
    route = router_forward(x_t[None, :], P["w_router"], P.get("router_bias"), top_k, renormalize)
    experts = route["expert_idx"][0] if forced_experts is None else np.asarray(forced_experts)
    sel = route["probs"][0, experts.astype(np.int64)]
    gates = sel / sel.sum() if renormalize else sel
    G = P["w_gate"] @ x_t
    U = P["w_up"] @ x_t
    y = np.zeros(P["w_down"].shape[0], F64)
    for j, e in enumerate(experts):
        e = int(e)
        a = G + s * (P["b_gate"][e] @ (P["a_gate"][e] @ x_t))
        b = U + s * (P["b_up"][e] @ (P["a_up"][e] @ x_t))
        h = silu(a) * b
        y += gates[j] * (P["w_down"] @ h + s * (P["b_down"][e] @ (P["a_down"][e] @ h)))
    return y, route


# --------------------------------------------------------------------------- #
# the block inside its transformer layer (Eq. 5 / Eq. 6)
# --------------------------------------------------------------------------- #
def rmsnorm(z, w_norm, eps):
    """LN of Eq. 5 for LLaMA-class models: root-mean-square normalisation over the model width with a learned
    per-channel weight (frozen here), `xn = w_norm * z / sqrt(mean(z^2) + eps)`.  Returns (xn [T, d], inv_rms [T])."""
    z = np.asarray(z, F64)
    inv_rms = 1.0 / np.sqrt(np.mean(z * z, axis=1) + eps)
    return z * inv_rms[:, None] * np.asarray(w_norm, F64)[None, :], inv_rms


def layer_forward(z, params, w_norm, eps, top_k, lora_alpha, renormalize=True, forced_expert_idx=None,
                  xn_round=None):
    """Eq. 6: `h = MixLoRA(LN(z)) + z`.  Returns (h [T, d], saved) where saved is that of `ffn_forward` on the
    normalised input plus `xn` and `inv_rms`.  `xn_round` (optional callable) is the rounding of the storage type
    in which an implementation keeps the normalised input: the router's discrete choice is then taken on the same
    values on both sides of a comparison."""
    xn, inv_rms = rmsnorm(z, w_norm, eps)
    if xn_round is not None:
        xn = np.asarray(xn_round(xn), F64)
    y, saved = ffn_forward(xn, params, top_k, lora_alpha, renormalize=renormalize,
                           forced_expert_idx=forced_expert_idx)
    saved = dict(saved)
    saved["xn"] = xn
    saved["inv_rms"] = inv_rms
    return np.asarray(z, F64) + y, saved


def layer_backward(z, params, w_norm, dh, saved, aux_coef=0.0, aux_f_mode=0, aux_batch=None):
    """Chain rule through Eq. 6.  `dh` = dL/dh.  The LoRA and router gradients are those of `ffn_backward` at the
    normalised input; `d_x` becomes dL/dz = dh (residual path) + the normalisation's Jacobian applied to dL/dxn:
    with `xh = z * inv_rms`, `u = dL/dxn * w_norm`:  `inv_rms * (u - xh * mean(u * xh))`."""
    z = np.asarray(z, F64)
    dh = np.asarray(dh, F64)
    g = ffn_backward(saved["xn"], params, dh, saved, aux_coef=aux_coef, aux_f_mode=aux_f_mode, want_dx=True,
                     aux_batch=aux_batch)
    inv_rms = saved["inv_rms"]
    xh = z * inv_rms[:, None]
    u = g["d_x"] * np.asarray(w_norm, F64)[None, :]
    g = dict(g)
    g["d_x"] = dh + inv_rms[:, None] * (u - xh * np.mean(u * xh, axis=1, keepdims=True))
    return g


# --------------------------------------------------------------------------- #
# plain LoRA on a linear layer (Eq. 1), as MixLoRA puts it on the attention projections (Section 3.2)
# --------------------------------------------------------------------------- #
def lora_linear_forward(x, w, a, b, lora_alpha):
    """`y = x W^T + s (x A^T) B^T`, `s = alpha / r`; W [out, in], A [r, in], B [out, r] (Eq. 1 applied to x)."""
    x, w, a, b = (np.asarray(v, F64) for v in (x, w, a, b))
    s = lora_alpha / a.shape[0]
    return x @ w.T + s * ((x @ a.T) @ b.T)


def lora_linear_backward(x, w, a, b, lora_alpha, dy):
    """Gradients of `<dy, y>`: W is frozen.  Returns dict(d_x, d_a, d_b)."""
    x, w, a, b, dy = (np.asarray(v, F64) for v in (x, w, a, b, dy))
    s = lora_alpha / a.shape[0]
    dz = s * (dy @ b)                       # [T, r]
    return dict(d_x=dy @ w + dz @ a, d_a=dz.T @ x, d_b=s * (dy.T @ (x @ a.T)))

