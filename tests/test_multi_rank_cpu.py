"""World-size-2 test of the cross-rank host logic of the benchmark (gloo, CPU only)."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent(
    """
    import os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_2002_11082_b200.sharding import worker_ids, max_over_ranks, aggregate_throughput
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ids = worker_ids(rank, 4)
    gathered = [None] * world
    dist.all_gather_object(gathered, ids)
    flat = sorted(i for g in gathered for i in g)
    assert flat == list(range(4 * world)), flat            # disjoint and complete
    ms = max_over_ranks(10.0 + 5.0 * rank, dist)            # rank 1 is the slow one
    assert ms == 15.0, ms
    assert abs(aggregate_throughput(3e9, ms, world) - 2 * 3e9 / 15e-3 / 1e9) < 1e-9
    # the data-parallel exchange: every rank ends up with every rank's codes and levels, in rank order
    import torch
    from paper_2002_11082_b200.sharding import CodeExchange
    words, T, s = 1000, 7, 9
    def codes_of(r): return (torch.arange(words, dtype=torch.int32) * 2654435 + 17 * r).remainder(100003)
    def levels_of(r): return torch.linspace(-1.0 - r, 1.0 + r, T * s).reshape(T, s)
    ex = CodeExchange(world, words, T, s)
    ex.gather(dist, codes_of(rank), levels_of(rank))
    for r in range(world):
        assert torch.equal(ex.all_packed[r], codes_of(r)), r
        assert torch.equal(ex.all_levels[r].reshape(T, s), levels_of(r)), r
    pk, lv = ex.pointer_rows()
    assert pk == [ex.all_packed.data_ptr() + 4 * words * r for r in range(world)]
    assert lv == [ex.all_levels.data_ptr() + 4 * T * s * r for r in range(world)]
    assert ex.recv_bytes == (world - 1) * 4 * (words + T * s)
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
    """
)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_gloo():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    from paper_2002_11082_b200.sharding import aggregate_throughput, max_over_ranks, worker_ids

    assert worker_ids(3, 8) == list(range(24, 32))
    assert max_over_ranks(7.5) == 7.5
    assert aggregate_throughput(1e9, 1.0, 1) == 1000.0
    import torch
    from paper_2002_11082_b200.sharding import CodeExchange

    ex = CodeExchange(1, 12, 2, 3)
    ex.gather(None, torch.arange(12, dtype=torch.int32), torch.arange(6, dtype=torch.float32).reshape(2, 3))
    assert ex.all_packed[0].tolist() == list(range(12)) and ex.recv_bytes == 0
    assert ex.pointer_rows() == ([ex.all_packed.data_ptr()], [ex.all_levels.data_ptr()])
