"""The N > 1 path of the benchmark on CPU (gloo, world size 2): every rank owns its own
batch of sequences (no collective on the data path), results are combined by a barrier and
a max-reduce of the elapsed time, and the whole-job value is the sum of the ranks' units
over that time."""
import os
import socket
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, q) -> None:
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from workloads import generate as gen, get_config
    base = get_config("c1")
    cfg = bench.rank_config(base, rank)
    # ranks work on different sequences: seeds, hence queries, differ
    q0 = gen.make_queries(cfg, 0, 1)
    sig = torch.tensor([float(q0.float().sum())])
    sigs = [torch.zeros(1) for _ in range(world)]
    dist.all_gather(sigs, sig)
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, device="cpu")
    value = bench.whole_job_value(world, steps=4, n_layers=cfg.n_layers, ms=ms)
    q.put((rank, cfg.seed, [float(x) for x in sigs], ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_take_the_max_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sigs0, ms0, v0), (r1, seed1, sigs1, ms1, v1) = res
    assert seed0 != seed1 and sigs0 == sigs1 and sigs0[0] != sigs0[1]
    assert ms0 == ms1 == 20.0                        # the slower rank's time, on both
    assert v0 == v1 == 2 * 4 * 1 / 20e-3             # both ranks' layer-steps over the max time


def test_cpulist_parser_and_numa_binding_falls_back_quietly():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.parse_cpulist("0-3,8,10-11\n") == {0, 1, 2, 3, 8, 10, 11}
    assert bench.parse_cpulist("5") == {5} and bench.parse_cpulist("") == set()
    before = os.sched_getaffinity(0)
    assert bench.bind_near_gpu(0) is None            # no GPU here: a placement hint must never raise
    assert os.sched_getaffinity(0) == before


def test_gpus_flag_starts_the_ranks_itself_when_no_launcher_set_the_environment():
    """`bench.py --gpus 2` with no WORLD_SIZE in the environment must come back as a two-rank job: the
    script re-executes itself under torch.distributed.run on 127.0.0.1 (checked here without a GPU: the
    ranks only call the roll, over gloo)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--launch-check"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                      # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ranks"] == [0, 1] and lines[0]["max_ms"] == 2.0
    # one rank needs no launcher
    r1 = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "1", "--launch-check"], env=env,
                        capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and json.loads(r1.stdout.strip().splitlines()[-1])["n_gpus"] == 1
