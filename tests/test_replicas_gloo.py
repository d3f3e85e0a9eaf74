"""The multi-GPU form of the benchmark is N independent replicas (the path has no exchange step).
World-size-2 check on CPU (gloo) of the only cross-rank logic there is: the job's time is the MAX over
ranks, the value is the whole-job aggregate, and the reference arm runs on rank 0 alone; plus the launch
path itself: `bench.py --gpus 2` started plainly starts two ranks, which rendezvous and report n_gpus 2."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 * (rank + 1)            # rank 1 is the slow replica
        ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
        value = bench.whole_job_gbs(step_bytes=5_000_000_000, steps=4, ms=ms, world=world)
        # identical seeded inputs on every replica: same lengths, same tables
        import ekv_inputs as I
        lengths = I.decode_lengths(I.C2)
        tables, _ = I.assign_blocks(I.C2.seed, 12, lengths, 16, 90000)
        digest = torch.tensor([int(lengths.sum()), int(tables.to(torch.int64).clamp(min=0).sum() % (1 << 40))])
        gathered = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(gathered, digest)
        with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
            f.write(f"{ms} {value} {int(all(torch.equal(g, digest) for g in gathered))}")
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_max_time_and_aggregate_value(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        ms, value, same = open(tmp_path / f"r{rank}.txt").read().split()
        assert float(ms) == 20.0                                         # max over ranks, on every rank
        assert abs(float(value) - 2 * 5.0 * 4 / 0.020) < 1e-6            # 2 replicas x 5 GB x 4 steps / 20 ms
        assert same == "1"


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench

    class Args:
        gpus, steps, warmup = 2, 1, 1
    monkeypatch.setenv("RANK", "1")
    assert bench.run_reference(Args) is None
    assert capsys.readouterr().out == ""


def test_bench_started_plainly_with_gpus_2_starts_two_ranks_itself():
    """No torchrun: bench.py spawns the ranks (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* as torchrun would set them).
    The GPU step is replaced by a host sleep of (rank + 1) x 20 ms (test hook --stub-ms) and the group runs on gloo;
    the reported time must be the slow rank's, the value the aggregate of both replicas."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "4", "--stub-ms", "20"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                                      # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["scaling"] == "weak"
    assert line["ms_per_step"] >= 40.0 > line["local_ms_rank0"] / 4      # the max over ranks, not rank 0's own time
    assert abs(line["value"] - 2 * 1.0 * 4 / (line["ms_per_step"] * 4 * 1e-3)) < 0.05 * line["value"]


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "1", "--stub-ms", "1"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "--gpus 4" in r.stderr
