"""The N > 1 plumbing of bench.py on CPU: two gloo ranks.  The path has no data-path collective
(every rank compresses its own replica of the workload); what the ranks share is the timing
reduction (a step costs what the slowest rank needs) and the rule that rank 0 alone reports."""
import io
import json
import os
import socket
import sys
from contextlib import redirect_stdout

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(1.0 + rank, dist, "cpu")          # rank r measured 1 + r ms
    dist.barrier()
    # the reference arm: rank 0 alone runs and prints, the others return without work
    buf = io.StringIO()
    sys.argv = ["bench.py", "--impl", "reference", "--gpus", str(world), "--steps", "1", "--warmup", "0",
                "--workload", "tiny"]
    with redirect_stdout(buf):
        bench.main()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"ms": ms, "stdout": buf.getvalue()}, f)
    dist.destroy_process_group()


def test_two_ranks_share_the_slowest_time_and_rank0_reports(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    assert [r["ms"] for r in res] == [2.0, 2.0]                  # max over ranks, on every rank
    assert res[1]["stdout"] == ""                                # only rank 0 prints
    line = json.loads(res[0]["stdout"])
    assert line["impl"] == "reference" and line["n_gpus"] == world and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
