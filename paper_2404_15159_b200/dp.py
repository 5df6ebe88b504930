"""Host-side helpers for data-parallel use of the block (one process per GPU, tokens sharded).

The block is row-wise independent, so ranks keep a full copy of the weights and their own
tokens; the only exchange of a training step is the sum of the LoRA and router gradients.
They are laid out in ONE flat fp32 buffer so that a single all-reduce covers them.
"""
from __future__ import annotations

GRAD_NAMES = ("d_a_gate", "d_b_gate", "d_a_up", "d_b_up", "d_a_down", "d_b_down", "d_w_router", "d_router_bias")


def grad_sizes(d_model: int, d_ff: int, n_experts: int, rank: int) -> dict:
    N, r, d, f = n_experts, rank, d_model, d_ff
    return {"d_a_gate": N * r * d, "d_b_gate": N * f * r, "d_a_up": N * r * d, "d_b_up": N * f * r,
            "d_a_down": N * r * f, "d_b_down": N * d * r, "d_w_router": N * d, "d_router_bias": N}


def flat_grad_layout(d_model: int, d_ff: int, n_experts: int, rank: int, align: int = 64):
    """(offsets, total): element offset of every gradient inside the flat buffer, each start a
    multiple of `align` elements (256 bytes) as the library wants 16-byte aligned outputs."""
    sizes = grad_sizes(d_model, d_ff, n_experts, rank)
    off, offsets = 0, {}
    for n in GRAD_NAMES:
        offsets[n] = (off, sizes[n])
        off += (sizes[n] + align - 1) // align * align
    return offsets, off


def shard_tokens(tokens: int, world: int, rank: int):
    """Contiguous token range [begin, end) of `rank` when `tokens` rows are split over `world` ranks."""
    base, rem = divmod(tokens, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
