"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank host logic: record sharding
and the whole-job rate (images of all ranks / slowest rank's time)."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 100.0 if rank == 0 else 250.0          # rank 1 is the slow one
    rate = bench.whole_job_rate(1024, 10, ms, world)
    mx = bench.reduce_max(ms, world)
    q.put((rank, bench.rank_record_index(rank), rate, mx))
    dist.destroy_process_group()


def test_two_ranks_shard_records_and_take_the_slowest_time():
    import torch.multiprocessing as mp
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [0, 1]                      # distinct records, no overlap
    for _, _, rate, mx in res:
        assert mx == 250.0
        assert rate == pytest.approx(2 * 1024 * 10 / 0.250)   # both ranks' images over the slowest time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, 1) == 3.5
    assert bench.whole_job_rate(100, 2, 50.0, 1) == pytest.approx(100 * 2 / 0.05)


def test_algorithmic_bytes_model():
    sys.path.insert(0, ROOT)
    import bench
    # one 32x32 image: 24 padded blocks, Y unpadded 16 blocks, chroma 4 each
    scans = [(3, 0, 0, 0, 0, 0, 100), (1, 0, 1, 5, 0, 0, 50), (1, 0, 1, 63, 2, 1, 70)]
    m = bench.algorithmic_bytes(scans, [(32, 32)], 3)
    assert m["clear"] == 128 * 24 and m["pixels"] == 128 * 24 + 3 * 1024
    assert m["index"] == 220
    assert m["entropy0"] == 100 + 2 * 1 * 24 + 50 + 2 * 5 * 16
    assert m["entropy1"] == 70 + 2 * 63 * 16 * 2
    m2 = bench.algorithmic_bytes(scans, [(32, 32)], 1)
    assert "entropy1" not in m2 and m2["index"] == 100
