"""Host logic of bench.py that needs no GPU: the max-over-ranks reduction used when every
rank decodes its own shard of lanes (world size 2, gloo), and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench.barrier(world)
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world)
    # lanes are sharded without overlap: rank r owns lanes [r*L, (r+1)*L)
    out[rank] = slowest
    dist.destroy_process_group()


def test_max_over_ranks_two_processes():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    assert out[0] == 15.0 and out[1] == 15.0


def test_reference_arm_prints_one_json_line():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--warmup", "3"], capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "logits/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                       capture_output=True, text=True, timeout=120, env=env)
    assert p.returncode == 0 and p.stdout.strip() == ""


def _gather_worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_2210_15458_b200 import shard
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_total, T = 7, 5                                   # 7 lanes over 2 ranks: shards of 4 and 3
    lo, hi = shard.shard_range(n_total, rank, world)
    full = torch.arange(n_total * T, dtype=torch.int32).reshape(n_total, T)
    lens = torch.arange(n_total, dtype=torch.int32) % (T + 1)
    seq, length = shard.gather_sequences(full[lo:hi].clone(), lens[lo:hi].clone(), n_total)
    out[rank] = (lo, hi, bool((seq == full).all()), bool((length == lens).all()))
    dist.destroy_process_group()


def test_lane_shards_and_the_final_gather_two_processes():
    sys.path.insert(0, ROOT)
    from paper_2210_15458_b200 import shard
    for n in (0, 1, 7, 64, 1000):
        for world in (1, 2, 3, 8):
            cuts = [shard.shard_range(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(cuts[r][1] == cuts[r + 1][0] for r in range(world - 1))
            sizes = [b - a for a, b in cuts]
            assert max(sizes) - min(sizes) <= 1
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_gather_worker, args=(2, 29741, out), nprocs=2, join=True)
    assert out[0] == (0, 4, True, True) and out[1] == (4, 7, True, True)


def _sharded_job_worker(rank, world, port, out):
    """The call sequence of a sharded decode, arguments only: shard_range -> the rank's
    as_step_lattice / as_decode_bigram arguments -> one gather at the end.  The kernels are
    replaced by the oracle's lattice codes and a deterministic stand-in for the sequences, so that
    what is checked is exactly what the sharding layer decides."""
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_2210_15458_b200 import shard
    from oracle import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, u, S, T = 37, 0.625, 5, 6
    # (a) one lattice sharded by lanes: the rank's slice of codes is the slice of the whole lattice
    a = shard.step_lattice_args(N, rank, world)
    whole = oracle.lattice_codes(N, u)
    mine = whole[a["j0"]: a["j0"] + a["lanes"]]                  # what as_step_lattice(j0, lanes) forms
    ok_codes = bool(np.array_equal(mine, oracle.lattice_codes(a["N"], u)[a["j0"]: a["j0"] + a["lanes"]]))
    # (b) a job of S start tokens x N codes sharded by start token, collected once at the end
    d = shard.decode_args(S, N, rank, world)
    starts = np.arange(100, 100 + S)

    def stand_in(start_tokens):                                   # lane = s*N + j -> a row that names (start, j)
        rows = [[int(s), j, 0, 0, 0, -1] for s in start_tokens for j in range(N)]
        return torch.tensor(rows, dtype=torch.int32).reshape(-1, T), torch.full((len(rows),), 5, dtype=torch.int32)
    seq, length = stand_in(starts[d["s_lo"]: d["s_hi"]])
    full_seq, full_len = shard.gather_sequences(seq, length, S * N, unit=N)
    want_seq, want_len = stand_in(starts)
    # contiguous lane blocks of the ranks tile the job: the gather of blocks of whole groups needs equal
    # lane counts per unit, which sharding by start token guarantees
    out[rank] = (a, d, ok_codes, bool((full_seq == want_seq).all()), bool((full_len == want_len).all()))
    dist.destroy_process_group()


def test_sharded_job_arguments_tile_the_single_rank_call():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_sharded_job_worker, args=(2, 29751, out), nprocs=2, join=True)
    a0, d0, c0, s0, l0 = out[0]
    a1, d1, c1, s1, l1 = out[1]
    assert c0 and c1 and s0 and s1 and l0 and l1
    assert a0["j0"] == 0 and a0["j0"] + a0["lanes"] == a1["j0"] and a1["j0"] + a1["lanes"] == 37
    assert d0["s_lo"] == 0 and d0["s_hi"] == d1["s_lo"] and d1["s_hi"] == 5
    assert d0["lane_hi"] == d1["lane_lo"] and d1["lane_hi"] == 5 * 37


def test_gpus_flag_must_match_the_ranks():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert p.returncode != 0 and "WORLD_SIZE" in (p.stderr + p.stdout)
