"""The multi-process path on CPU: two gloo ranks shard utterances, run the (CPU) stand-in for
the per-rank work, and combine timing (max) and unit counts (sum) the way bench.py does."""
import os
import subprocess
import sys
import textwrap

from paper_2603_11243_b200 import dist as D

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_partition_by_bytes_is_contiguous_and_balanced():
    costs = [5, 1, 1, 1, 8, 2, 2, 4, 4, 4]
    for world in (1, 2, 3, 4, 10, 13):
        parts = D.partition_by_bytes(costs, world)
        assert len(parts) == world
        assert parts[0][0] == 0 and parts[-1][1] == len(costs)
        for (a, b), (c, d) in zip(parts, parts[1:]):
            assert b == c and a <= b
        if world <= 4:
            loads = [sum(costs[a:b]) for a, b in parts]
            assert max(loads) <= sum(costs) / world + max(costs)
    assert D.partition_by_bytes([], 3) == [(0, 0)] * 3


def test_vocab_shards_tile_the_vocabulary():
    for V in (1, 7, 8, 9, 1001, 49152, 152064):
        for world in (1, 2, 3, 8):
            spans = [D.vocab_shard(V, r, world) for r in range(world)]
            at = 0
            for col0, n in spans:
                assert n >= 0 and (n == 0 or col0 == at)
                at += n
            assert at == V
            assert all(col0 % 8 == 0 for col0, n in spans if n)


def test_all_gather_rows_without_a_process_group():
    import torch
    x = torch.arange(6.0).reshape(2, 3)
    assert torch.equal(D.all_gather_rows(x), x.unsqueeze(0))


def test_rank_seeds_differ_and_rank0_keeps_the_workload_seed():
    assert D.rank_seed(7, 0) == 7
    assert len({D.rank_seed(7, r) for r in range(8)}) == 8


WORKER = textwrap.dedent("""
    import sys, torch
    sys.path.insert(0, %r)
    from paper_2603_11243_b200 import dist as D
    from paper_2603_11243_b200 import synth
    rank, local_rank, world = D.init("gloo")
    assert world == 2
    # every rank draws its own batch of the workload (weak scaling): different seeds, same shape
    w = synth.scaled(synth.CONFIGS[1], B=4, seed=D.rank_seed(synth.CONFIGS[1].seed, rank))
    T = synth.draw_lengths(w)
    gathered = [None, None]
    torch.distributed.all_gather_object(gathered, T)
    assert gathered[0] != gathered[1], "ranks must not process the same utterances"
    D.barrier()
    ms_max, units = D.reduce_max_sum(10.0 + 5.0 * rank, float(w.B), "cpu")
    assert ms_max == 15.0 and units == 8.0, (ms_max, units)
    # a given batch split by bytes: the two ranges are disjoint and cover it
    costs = [t * w.V_ctc * 2 for t in gathered[0]]
    lo, hi = D.partition_by_bytes(costs, world)[rank]
    spans = [None, None]
    torch.distributed.all_gather_object(spans, (lo, hi))
    assert spans[0][1] == spans[1][0] and spans[0][0] == 0 and spans[1][1] == len(costs)
    # the exchange of vocabulary-parallel verification: every rank's [M, 3] statistics, rank-major
    V_total = 1001
    col0, v_local = D.vocab_shard(V_total, rank, world)
    mine = torch.full((5, 3), float(rank)) + torch.arange(15.0).reshape(5, 3) / 100
    mine[:, 2] = col0
    allr = D.all_gather_rows(mine)
    assert tuple(allr.shape) == (2, 5, 3) and allr.is_contiguous()
    assert torch.equal(allr[rank], mine) and allr[1 - rank][0, 0] == float(1 - rank)
    assert allr[0][0, 2] == 0 and allr[1][0, 2] == D.vocab_shard(V_total, 1, world)[0]
    D.finalize()
    sys.stdout.write("rank%%d-ok\\n" %% rank)
""")


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                        "--nproc-per-node", "2", "--master-addr", "127.0.0.1", "--master-port",
                        "29541", str(script)], capture_output=True, text=True, timeout=240, env=env)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "rank0-ok" in r.stdout and "rank1-ok" in r.stdout
