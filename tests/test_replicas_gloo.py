"""Host logic of the multi-GPU bench path, run as two gloo ranks on CPU: the path does not shard
(replicas only), so the only exchange is the max-over-ranks of the step time."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 2.0 + 3.0 * rank          # rank 1 is the slow one
    dist.barrier()
    ms_max, value = bench.aggregate_replicas(ms_local, step_bytes=10 ** 9, world=world, device="cpu")
    out[rank] = (ms_max, value, bench.replica_seed(rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for rank in range(world):
        ms_max, value, _ = out[rank]
        assert ms_max == 5.0
        # two replicas x 1 GB per step in 5 ms = 400 GB/s
        assert abs(value - 400.0) < 1e-9
    assert out[0][2] != out[1][2]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms_max, value = bench.aggregate_replicas(4.0, step_bytes=2 * 10 ** 9, world=1, device="cpu")
    assert ms_max == 4.0 and abs(value - 500.0) < 1e-9


def test_gpus_flag_without_a_launcher_starts_one_rank_per_gpu():
    """`bench.py --gpus N` with no WORLD_SIZE in the environment re-executes itself under torch.distributed.run with
    N ranks on 127.0.0.1; the command keeps the caller's flags. The reference arm is used to run it for real on CPU:
    rank 0 prints the line, the other rank exits 0 without work."""
    import json
    import subprocess
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launch_command(4, ["--gpus", "4", "--steps", "7"], port=12345)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "12345" and cmd[-4:] == ["--gpus", "4", "--steps", "7"]
    assert cmd[-5].endswith("bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
