"""The N > 1 path of the benchmark on CPU with gloo, world size 2: the path shards over tokens with no
data-path collective, so the only cross-rank step is the MAX reduction of the step time; each rank draws its
own seeded inputs; the reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    import synth_inputs as si
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(3.0 + rank, world)              # rank 1 is the slow one
    x = si.channel_scaled_activation(32, 64, seed=rank * 3 + 1)
    gathered = [torch.zeros_like(x) for _ in range(world)]
    dist.all_gather(gathered, x)                               # test-only exchange, to compare the shards
    out[rank] = (ms, bench.job_value(ms, world), bool(torch.equal(gathered[0], gathered[1])))
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_value():
    import bench
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 4.0                       # the slowest rank's time, on every rank
    assert res[0][1] == 2 * bench.FLOPS_PER_STEP / 4.0e-3 / 1e12
    assert res[0][2] is False                                  # ranks work on different tokens
    assert bench.max_over_ranks(5.0, 1) == 5.0


def test_reference_arm_prints_from_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def _amax_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2609_02846_b200.autograd import reduce_amax_
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t = torch.tensor([1.5 + 2.0 * rank])                      # each rank sampled its own shard's maximum
    reduce_amax_(t, dist.group.WORLD)
    out[rank] = float(t.item())
    dist.destroy_process_group()


def test_refresh_step_amax_is_agreed_across_ranks():
    """On refresh steps the sampled maxima are MAX-all-reduced (one float per operand): the only exchange of the path."""
    port = 31500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_amax_worker, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0] == res[1] == 3.5


def test_layers_ranks_and_steps_draw_from_different_streams():
    """Eq. "sr" assumes independent draws: the base seed of a backward pass differs between two layers built with the
    default seed, between two data-parallel ranks and between two steps, and so do the 16-bit draws the oracle's
    generator gives for the same element index; both quantizations of dY inside one pass (4s and 4s + 1) differ too."""
    import oracle
    from paper_2609_02846_b200 import autograd
    a = autograd.Ue5m3Linear(256, 256, device="cpu")
    b = autograd.Ue5m3Linear(256, 256, device="cpu")
    assert a.seed != b.seed and a.rank == b.rank == 0
    seeds = {autograd.sr_stream_seed(layer, rank, step) for layer in (a.seed, b.seed) for rank in (0, 1, 7) for step in (0, 1, 50)}
    assert len(seeds) == 18 and max(seeds) < 2 ** 62
    streams = set()
    for s in seeds:
        for role in (0, 1):
            streams.add(tuple(oracle.sr_bits(4 * s + role, i) for i in range(16)))
    assert len(streams) == 36


def _rank_seed_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2609_02846_b200 import autograd
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layer = autograd.Ue5m3Linear(256, 256, device="cpu", seed=5, group=dist.group.WORLD)
    out[rank] = (layer.rank, autograd.sr_stream_seed(layer.seed, layer.rank, 3))
    dist.destroy_process_group()


def test_rank_is_mixed_into_the_gradient_draws():
    port = 33500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_seed_worker, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0][0] == 0 and res[1][0] == 1 and res[0][1] != res[1][1]
