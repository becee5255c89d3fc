"""The multi-GPU path is independent replicas; its host logic (sharding, max-over-ranks timing, summed tokens)
is exercised here with two gloo ranks on the CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_range_covers_everything():
    from paper_2605_01106_b200.replicas import shard_range
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in shard_range(n, r, world)]
            assert got == list(range(n))
            sizes = [len(shard_range(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_two_gloo_ranks_aggregate():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = textwrap.dedent("""
        import os, sys
        sys.path.insert(0, %r)
        import torch.distributed as dist
        from paper_2605_01106_b200.replicas import shard_range, reduce_max_sum, job_throughput
        dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d", rank=int(os.environ["RANK"]), world_size=2)
        rank = dist.get_rank()
        mine = shard_range(5, rank, 2)                       # 3 + 2 sequences
        ms, toks = reduce_max_sum(10.0 + 5.0 * rank, 100.0 * len(mine), 2)
        assert ms == 15.0 and toks == 500.0, (ms, toks)
        assert abs(job_throughput(10.0 + 5.0 * rank, 100.0 * len(mine), 2) - 500.0 / 15e-3) < 1e-6
        dist.barrier()
        dist.destroy_process_group()
        print("rank", rank, "ok")
    """) % (ROOT, port)
    procs = [subprocess.Popen([sys.executable, "-c", code], env={**os.environ, "RANK": str(r)},
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out
