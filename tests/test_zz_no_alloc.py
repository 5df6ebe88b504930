"""The workspace-free dispatch entry point against the regular one.

`mixlora_dispatch_static` exists for callers that cannot allocate device memory (they have
no workspace to hand over); its scratch is a fixed array inside the library.  Here it is
called through the C ABI twice in a row - a larger problem first, then a smaller one, so that
anything the first call left in the shared scratch would show - and its outputs must equal,
bit for bit, the permutation and segment offsets that `mixlora_ffn_forward` produces for the
same routing.  The file name makes pytest collect it last.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import mixlora_oracle as orc
from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu


def _routing_from_forward(B, torch, w):
    t = synth.generate(w, with_dy=False)
    act = torch.float32
    dev = {n: (None if v is None else torch.from_numpy(v).cuda().to(act if n not in ("w_router", "router_bias") else torch.float32))
           for n, v in t.items()}
    shape = B.make_shape(w.tokens, w.d_model, w.d_ff, w.n_experts, w.top_k, w.rank, w.lora_alpha, B.MIXLORA_DTYPE_FP32)
    params = B.make_params(**{n: dev[n] for n in synth.PARAM_NAMES}, x=dev["x"])
    ws = B.alloc_workspace(shape, False)
    y = torch.empty(w.tokens, w.d_model, dtype=act, device="cuda")
    B.mixlora_ffn_forward(shape, params, y, ws)
    torch.cuda.synchronize()
    view = B.mixlora_routing_view(shape, ws)
    return {n: v.clone() for n, v in view.items()}


def test_static_dispatch_matches_the_workspace_path_on_two_calls_in_a_row():
    import torch
    from paper_2404_15159_b200 import binding as B

    base = dict(d_model=64, d_ff=128, rank=8, lora_alpha=16.0, dtype="fp32", std_frozen=0.05, std_a=0.05, std_b=0.05)
    cases = [synth.Workload("static-a", tokens=3000, n_experts=16, top_k=3, seed=synth.BASE_SEED + 200, **base),
             synth.Workload("static-b", tokens=517, n_experts=5, top_k=2, seed=synth.BASE_SEED + 201, **base)]
    refs = [_routing_from_forward(B, torch, w) for w in cases]
    # outputs are allocated before the calls under test; the calls themselves allocate nothing
    outs = [(torch.full((w.tokens * w.top_k,), -1, dtype=torch.int32, device="cuda"),
             torch.full((w.n_experts + 1,), -1, dtype=torch.int32, device="cuda")) for w in cases]
    for w, ref, (perm, seg_off) in zip(cases, refs, outs):          # two calls in a row, same stream
        B.mixlora_dispatch_static(ref["expert_idx"], w.tokens, w.n_experts, w.top_k, perm, seg_off)
    torch.cuda.synchronize()
    for w, ref, (perm, seg_off) in zip(cases, refs, outs):
        assert torch.equal(perm, ref["perm"]), w.name
        assert torch.equal(seg_off, ref["seg_off"]), w.name
        assert sorted(perm.cpu().tolist()) == list(range(w.tokens * w.top_k))
        want = orc.dispatch(ref["expert_idx"].cpu().numpy(), w.n_experts)        # and the oracle's dispatch directly
        np.testing.assert_array_equal(perm.cpu().numpy(), want["perm"])
        np.testing.assert_array_equal(seg_off.cpu().numpy(), want["seg_off"])


def test_static_dispatch_at_its_stated_maximum_and_with_the_larger_problem_second():
    # 65536 tokens, 32 experts, top-8: the whole fixed scratch is in use (256 blocks x 32 experts, both tables).
    # A small problem runs first on the same stream, so the large one starts from a scratch that holds leftovers.
    import torch
    from paper_2404_15159_b200 import binding as B

    rng = np.random.default_rng(7)
    cases = []
    for tokens, N, k in ((700, 6, 3), (B.mixlora_dispatch_static_max_tokens(), 32, 8)):
        keys = rng.random((tokens, N))
        idx = np.argsort(keys, axis=1)[:, :k].astype(np.int32)                  # k distinct experts per token
        cases.append((tokens, N, k, idx))
    outs = []
    for tokens, N, k, idx in cases:
        dev_idx = torch.from_numpy(idx).cuda()
        perm = torch.full((tokens * k,), -1, dtype=torch.int32, device="cuda")
        seg = torch.full((N + 1,), -1, dtype=torch.int32, device="cuda")
        outs.append((dev_idx, perm, seg))
    for (tokens, N, k, idx), (dev_idx, perm, seg) in zip(cases, outs):
        B.mixlora_dispatch_static(dev_idx, tokens, N, k, perm, seg)
    torch.cuda.synchronize()
    for (tokens, N, k, idx), (dev_idx, perm, seg) in zip(cases, outs):
        flat = idx.reshape(-1)
        want_perm = np.argsort(flat, kind="stable").astype(np.int32)            # expert ascending, slot ascending
        want_seg = np.concatenate([[0], np.cumsum(np.bincount(flat, minlength=N))]).astype(np.int32)
        np.testing.assert_array_equal(perm.cpu().numpy(), want_perm)
        np.testing.assert_array_equal(seg.cpu().numpy(), want_seg)


def test_static_dispatch_skips_indices_outside_the_expert_range():
    import torch
    from paper_2404_15159_b200 import binding as B

    idx = np.array([[0, 1], [2, 9], [-3, 1], [1, 0]], np.int32)               # 9 and -3 are not experts of N = 3
    dev_idx = torch.from_numpy(idx).cuda()
    perm = torch.full((8,), -1, dtype=torch.int32, device="cuda")
    seg = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    B.mixlora_dispatch_static(dev_idx, 4, 3, 2, perm, seg)
    torch.cuda.synchronize()
    assert seg.cpu().tolist() == [0, 2, 5, 6]
    assert perm.cpu().tolist() == [0, 7, 1, 5, 6, 2, -1, -1]                   # skipped slots leave the tail untouched


def test_static_dispatch_rejects_sizes_beyond_its_fixed_scratch():
    import torch
    from paper_2404_15159_b200 import binding as B

    limit = B.mixlora_dispatch_static_max_tokens()
    assert limit == 65536
    buf = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MixLoraError) as err:
        B.mixlora_dispatch_static(buf, limit + 1, 8, 2, buf, buf)
    assert err.value.status == 2
    with pytest.raises(B.MixLoraError) as err:
        B.mixlora_dispatch_static(buf, 16, 64, 2, buf, buf)
    assert err.value.status == 2
    with pytest.raises(B.MixLoraError) as err:
        B.mixlora_dispatch_static(None, 16, 8, 2, buf, buf)
    assert err.value.status == 1
    seg = torch.full((9,), 7, dtype=torch.int32, device="cuda")
    B.mixlora_dispatch_static(buf, 0, 8, 2, buf, seg)                # zero tokens: offsets all zero
    assert int(seg.abs().sum().item()) == 0
