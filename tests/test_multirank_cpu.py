"""The N > 1 host logic on CPU: two gloo ranks shard the sequences, draw distinct inputs
and reduce their timings to the whole-job figure the benchmark prints."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_13204_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.scaled(synth.workload(4), batch=6, prompt_len=64)
        mine = shard.rank_sequences(w.batch, world, rank)
        seed = shard.rank_seed(w.seed, rank)
        prompts = [synth.prompt_ids(synth.scaled(w, seed=seed), b) for b in range(w.batch)]
        digest = int(torch.cat(prompts).to(torch.int64).sum().item())
        # every rank sees every rank's block and digest
        got = [None] * world
        dist.all_gather_object(got, (list(mine), seed, digest))
        ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
        ms_max = shard.max_over_ranks(ms)
        rate = shard.whole_job_rate(units_per_rank_per_step=w.rows_per_step, steps=4, world=world, ms_max=ms_max)
        if rank == 0:
            out.put((got, ms_max, rate, w.rows_per_step))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_reduce_timing():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got, ms_max, rate, rows = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    blocks = [set(g[0]) for g in got]
    assert blocks[0].isdisjoint(blocks[1]) and sorted(blocks[0] | blocks[1]) == list(range(12))
    assert got[0][1] != got[1][1] and got[0][2] != got[1][2]      # distinct seeds, distinct inputs
    assert ms_max == 15.0                                         # the slowest rank sets the time
    assert rate == world * rows * 4 / 15.0e-3


def test_single_process_needs_no_group():
    assert shard.max_over_ranks(3.5) == 3.5
    assert list(shard.rank_sequences(4, 1, 0)) == [0, 1, 2, 3]
    assert shard.rank_seed(4, 0) == 4


def test_launch_plan():
    assert shard.launch_plan(1, {}) == "run"
    assert shard.launch_plan(4, {}) == "spawn"
    assert shard.launch_plan(4, {"WORLD_SIZE": "4"}) == "run"
    assert shard.launch_plan(1, {"WORLD_SIZE": "1"}) == "run"
    for bad in ((2, {"WORLD_SIZE": "4"}), (1, {"WORLD_SIZE": "2"}), (0, {})):
        try:
            shard.launch_plan(*bad)
        except ValueError:
            continue
        raise AssertionError(bad)


_RANK_SCRIPT = """
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
from paper_2505_13204_b200 import shard
assert shard.launch_plan(int(sys.argv[1])) == "run"
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = shard.max_over_ranks(7.0 + rank)
if rank == 0:
    print(json.dumps({"n_gpus": world, "ms": ms, "seed": shard.rank_seed(4, rank)}))
dist.destroy_process_group()
"""


def test_spawned_ranks_form_a_group_of_the_size_asked_for(tmp_path, capfd):
    """The launcher path of `bench.py --gpus N` (started plainly, N > 1): the program starts N
    ranks of itself; every rank sees the group, rank 0 prints the line."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "rank_script.py"
    script.write_text(_RANK_SCRIPT % root)
    rc = shard.spawn_ranks(str(script), ["2"], 2, extra_env={"OMP_NUM_THREADS": "1"})
    out = capfd.readouterr().out
    assert rc == 0
    import json
    line = [json.loads(l) for l in out.splitlines() if l.startswith("{")][-1]
    assert line == {"n_gpus": 2, "ms": 8.0, "seed": 4}
