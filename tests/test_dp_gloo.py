"""Data-parallel host logic on CPU ranks (gloo, world size 2): sharding of tokens and the single
all-reduce of the flat gradient buffer.  Each rank runs the CPU oracle on its shard; the summed
gradients must equal the full-batch oracle gradients (the main loss is a sum over tokens; the
auxiliary loss is per shard by design, so it is switched off here)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import mixlora_oracle as orc
    from paper_2404_15159_b200 import dp, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.Workload("dp", tokens=37, d_model=16, d_ff=24, n_experts=4, top_k=2, rank=4, lora_alpha=8.0, dtype="fp32",
                       std_frozen=0.3, std_a=0.3, std_b=0.3, seed=synth.BASE_SEED + 300)
    t = synth.generate(w)
    b, e = dp.shard_tokens(w.tokens, world, rank)
    params = synth.params_of(t)
    _, saved = orc.ffn_forward(t["x"][b:e], params, w.top_k, w.lora_alpha)
    g = orc.ffn_backward(t["x"][b:e], params, t["dy"][b:e], saved, aux_coef=0.0, want_dx=False)
    offsets, total = dp.flat_grad_layout(w.d_model, w.d_ff, w.n_experts, w.rank)
    flat = torch.zeros(total, dtype=torch.float64)
    for n, (off, size) in offsets.items():
        flat[off:off + size] = torch.from_numpy(np.ascontiguousarray(g[n]).reshape(-1))
    dist.all_reduce(flat)
    if rank == 0:
        np.save(os.path.join(out_dir, "flat.npy"), flat.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_gradients_sum_to_the_full_batch_gradients(tmp_path):
    from oracle import mixlora_oracle as orc
    from paper_2404_15159_b200 import dp, synth
    world = 2
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    flat = np.load(tmp_path / "flat.npy")
    w = synth.Workload("dp", tokens=37, d_model=16, d_ff=24, n_experts=4, top_k=2, rank=4, lora_alpha=8.0, dtype="fp32",
                       std_frozen=0.3, std_a=0.3, std_b=0.3, seed=synth.BASE_SEED + 300)
    t = synth.generate(w)
    params = synth.params_of(t)
    _, saved = orc.ffn_forward(t["x"], params, w.top_k, w.lora_alpha)
    g = orc.ffn_backward(t["x"], params, t["dy"], saved, aux_coef=0.0, want_dx=False)
    offsets, total = dp.flat_grad_layout(w.d_model, w.d_ff, w.n_experts, w.rank)
    assert flat.shape == (total,)
    for n, (off, size) in offsets.items():
        np.testing.assert_allclose(flat[off:off + size], np.asarray(g[n]).reshape(-1), rtol=1e-10, atol=1e-12, err_msg=n)


def test_shards_cover_every_token_once_and_offsets_are_aligned():
    from paper_2404_15159_b200 import dp
    for tokens in (0, 1, 7, 8192, 8193):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                b, e = dp.shard_tokens(tokens, world, r)
                assert 0 <= b <= e <= tokens
                seen.extend(range(b, e))
            assert seen == list(range(tokens))
    offsets, total = dp.flat_grad_layout(4096, 11008, 8, 16)
    sizes = dp.grad_sizes(4096, 11008, 8, 16)
    end = 0
    for n in dp.GRAD_NAMES:
        off, size = offsets[n]
        assert off % 64 == 0 and off >= end and size == sizes[n]
        end = off + size
    assert total >= end
