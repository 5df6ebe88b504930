"""Data-parallel host logic on CPU ranks (gloo, world size 2): sharding of tokens, the all-reduce of the 2N
auxiliary-loss sums (Eq. 8-9 are fractions of the whole batch) and the single all-reduce of the flat gradient
buffer.  Each rank runs the CPU oracle on its shard; the summed gradients must equal the full-batch oracle
gradients, auxiliary loss included.  Also: `bench.py --gpus 2` started without a launcher starts its own ranks."""
import json
import subprocess
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
AUX_COEF = 0.4


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
    # exchange 1: the shards' un-normalised sums of Eq. 9 (2N numbers), as the library's mixlora_aux_stats /
    # mixlora_aux_loss_global pair is used
    count, psum = orc.aux_sums(saved["route"]["probs"], saved["route"]["expert_idx"])
    sums = torch.from_numpy(np.concatenate([psum, count]))
    dist.all_reduce(sums)
    loss, F, _ = orc.aux_loss_from_sums(sums[w.n_experts:].numpy(), sums[:w.n_experts].numpy(), w.tokens, w.top_k,
                                        AUX_COEF)
    g = orc.ffn_backward(t["x"][b:e], params, t["dy"][b:e], saved, aux_coef=AUX_COEF, want_dx=False,
                         aux_batch=(F, w.tokens))
    offsets, total = dp.flat_grad_layout(w.d_model, w.d_ff, w.n_experts, w.rank)
    flat = torch.zeros(total, dtype=torch.float64)
    for n, (off, size) in offsets.items():
        flat[off:off + size] = torch.from_numpy(np.ascontiguousarray(g[n]).reshape(-1))
    dist.all_reduce(flat)
    if rank == 0:
        np.save(os.path.join(out_dir, "flat.npy"), flat.numpy())
        np.save(os.path.join(out_dir, "loss.npy"), np.array([loss]))
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
    g = orc.ffn_backward(t["x"], params, t["dy"], saved, aux_coef=AUX_COEF, want_dx=False)
    full_loss, _, _ = orc.aux_loss(saved["route"]["probs"], saved["route"]["expert_idx"], AUX_COEF)
    assert float(np.load(tmp_path / "loss.npy")[0]) == pytest.approx(full_loss, rel=1e-12)
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


def test_bench_started_without_a_launcher_starts_its_own_ranks():
    # `python bench.py --gpus 2` with no WORLD_SIZE in the environment must become two ranks and report n_gpus = 2;
    # --stub keeps the ranks on the CPU (gloo) around a stand-in step, the launch path is the one the CUDA leg uses
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub", "--steps", "4",
                        "--warmup", "3"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["warmup"] == 3
    assert line["config"]["parallelism"].startswith("dp2")
