"""The multi-GPU form of the benchmark is N independent replicas (the path has no exchange step).
World-size-2 check on CPU (gloo) of the only cross-rank logic there is: the job's time is the MAX over
ranks, the value is the whole-job aggregate, and the reference arm runs on rank 0 alone."""
import os
import socket
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
