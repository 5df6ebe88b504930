"""Seeded synthetic inputs shaped like the paper's LLaMA-class fine-tuning workloads.

This module only draws random tensors and rounds them to the storage type; it
holds none of the method's arithmetic, so both the CUDA path and the CPU oracle
may be fed from it.  All draws come from numpy's counter-based Philox generator.

Shapes follow Table 3 of the paper (8 experts, top-2, rank 16, alpha 32 on the
gate / up / down projections) applied to the LLaMA-2 7B and 13B FFN sizes; the
second argument of every N(., .) below is a standard deviation.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 0x4D49584C


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    rank: int
    lora_alpha: float
    dtype: str            # "bf16" or "fp32"
    std_frozen: float
    std_a: float
    std_b: float
    zipf_s: float = 0.0   # > 0: router bias so that expert shares are Zipf-like
    seed: int = BASE_SEED

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def c1() -> Workload:
    return Workload("C1-tiny-fp32", 256, 256, 688, 4, 2, 8, 16.0, "fp32", 0.02, 0.02, 0.02, seed=BASE_SEED + 0)


def c2() -> Workload:
    return Workload("C2-llama2-7b-fwd", 4096, 4096, 11008, 8, 2, 16, 32.0, "bf16", 0.02, 1.0 / 16, 0.01,
                    seed=BASE_SEED + 1)


def c3() -> Workload:
    return Workload("C3-llama2-7b-train", 8192, 4096, 11008, 8, 2, 16, 32.0, "bf16", 0.02, 1.0 / 16, 0.01,
                    seed=BASE_SEED + 2)


def c4() -> Workload:
    return Workload("C4-llama2-13b-train", 8192, 5120, 13824, 8, 2, 16, 32.0, "bf16", 0.02, 1.0 / 16, 0.01,
                    seed=BASE_SEED + 3)


def c5(n_experts: int, top_k: int, rank: int, tokens: int) -> Workload:
    return Workload(f"C5-zipf-N{n_experts}-k{top_k}-r{rank}-T{tokens}", tokens, 4096, 11008, n_experts, top_k,
                    rank, 2.0 * rank, "bf16", 0.02, 1.0 / rank, 0.01, zipf_s=1.2, seed=BASE_SEED + 4)


def llama3_8b(tokens: int = 8192) -> Workload:
    """Second workload shape: LLaMA-3-8B's FFN (d = 4096, f = 14336), same adapter set-up as c3."""
    return Workload(f"llama3-8b-T{tokens}", tokens, 4096, 14336, 8, 2, 16, 32.0, "bf16", 0.02, 1.0 / 16, 0.01,
                    seed=BASE_SEED + 5)


def wide_2b(tokens: int = 8192) -> Workload:
    """Second workload shape: a 2B-class model with a wide FFN (d = 2048, f = 16384; the width ratio of Gemma-2B,
    with the SwiGLU activation of this block)."""
    return Workload(f"wide-2b-T{tokens}", tokens, 2048, 16384, 8, 2, 16, 32.0, "bf16", 0.02, 1.0 / 16, 0.01,
                    seed=BASE_SEED + 6)


def c5_grid():
    return [c5(n, k, r, t) for n in (8, 16) for k in (1, 2) for r in (8, 16, 64) for t in (512, 4096, 32768)]


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable float32."""
    return (np.ascontiguousarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)


def zipf_bias(w: Workload) -> np.ndarray:
    """Router bias that skews expert selection towards q_i proportional to i^-s.

    With logits of standard deviation sigma = std_frozen * sqrt(d) (x ~ N(0,1)),
    adding beta * log q_i with beta = sigma * sqrt(6) / pi (the scale of a Gumbel
    variable of the same spread) makes the arg-max shares roughly q_i.  It is a
    recipe for skewed load, not a fit; the achieved shares are reported by the
    caller.
    """
    q = np.arange(1, w.n_experts + 1, dtype=np.float64) ** (-w.zipf_s)
    q /= q.sum()
    sigma = w.std_frozen * math.sqrt(w.d_model)
    beta = sigma * math.sqrt(6.0) / math.pi
    b = beta * np.log(q)
    return (b - b.mean()).astype(np.float32)


def generate(w: Workload, with_dy: bool = True) -> dict:
    """All tensors of one workload as float32 numpy arrays.

    For bf16 workloads every tensor except the router (fp32 by design) is rounded
    to bf16 once, here, so both sides see identical values.
    """
    rng = np.random.Generator(np.random.Philox(key=w.seed))
    T, d, f, N, r = w.tokens, w.d_model, w.d_ff, w.n_experts, w.rank

    def normal(shape, std):
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(std)

    t = {}
    # weights first, so that a workload with fewer tokens keeps the same weights
    t["w_gate"] = normal((f, d), w.std_frozen)
    t["w_up"] = normal((f, d), w.std_frozen)
    t["w_down"] = normal((d, f), w.std_frozen)
    t["w_router"] = normal((N, d), w.std_frozen)
    t["a_gate"] = normal((N, r, d), w.std_a)
    t["b_gate"] = normal((N, f, r), w.std_b)
    t["a_up"] = normal((N, r, d), w.std_a)
    t["b_up"] = normal((N, f, r), w.std_b)
    t["a_down"] = normal((N, r, f), w.std_a)
    t["b_down"] = normal((N, d, r), w.std_b)
    t["x"] = normal((T, d), 1.0)
    if with_dy:
        t["dy"] = normal((T, d), 1.0)
    t["router_bias"] = zipf_bias(w) if w.zipf_s > 0 else None
    if w.dtype == "bf16":
        for n in list(t):
            if n in ("w_router", "router_bias") or t[n] is None:
                continue
            t[n] = round_to_bf16(t[n])
    return t


PARAM_NAMES = ("w_gate", "w_up", "w_down", "w_router", "router_bias",
               "a_gate", "b_gate", "a_up", "b_up", "a_down", "b_down")


def params_of(tensors: dict) -> dict:
    return {n: tensors[n] for n in PARAM_NAMES}
