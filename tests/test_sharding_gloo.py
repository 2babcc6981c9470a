"""The multi-rank path on CPU: rows are independent, so N ranks shard the batch
with no data-path collective.  Two gloo ranks each take their block of rows,
and the gathered per-token results must equal the single-rank results; the
benchmark's max-over-ranks reduction is exercised the same way."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2512_23087_b200 import inputs


def test_shard_rows_covers_every_row_once():
    for T in (0, 1, 7, 64, 1000, 32768):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                r0, r1 = inputs.shard_rows(T, r, world)
                assert 0 <= r0 <= r1 <= T
                seen.extend(range(r0, r1))
            assert seen == list(range(T))


def _bits(x):
    return x.view(torch.int16).numpy().view(np.uint16)


def _worker(rank, world, port, T, V, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.WORKLOADS["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=3, device="cpu", T=T, V=V)      # same seed: same batch everywhere
    r0, r1 = inputs.shard_rows(T, rank, world)
    res = oracle.dvp_rows(_bits(batch.train[r0:r1]), batch.ids[r0:r1].numpy(), 1e-3, dtype=oracle.BF16,
                          infer=_bits(batch.infer[r0:r1]))
    per = (T + world - 1) // world
    local = torch.full((per, 3), float("nan"), dtype=torch.float64)
    local[: r1 - r0, 0] = torch.from_numpy(res.train.logp_mp)
    local[: r1 - r0, 1] = torch.from_numpy(res.log_ratio)
    local[: r1 - r0, 2] = torch.from_numpy(res.train.count.astype(np.float64))
    gathered = [torch.empty_like(local) for _ in range(world)]
    dist.all_gather(gathered, local)
    # the benchmark's reduction: device time of the job = max over ranks
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        torch.save({"rows": torch.cat(gathered)[:T], "t_max": t.item()}, os.path.join(out_dir, "out.pt"))
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_rank_result(tmp_path):
    T, V, world = 37, 3000, 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, T, V, str(tmp_path)), nprocs=world, join=True)
    got = torch.load(os.path.join(tmp_path, "out.pt"))
    w = inputs.WORKLOADS["c2_bf16_fwdbwd"]
    batch = inputs.make_rows(w, seed=3, device="cpu", T=T, V=V)
    want = oracle.dvp_rows(_bits(batch.train), batch.ids.numpy(), 1e-3, dtype=oracle.BF16,
                           infer=_bits(batch.infer))
    rows = got["rows"].numpy()
    assert np.array_equal(rows[:, 0], want.train.logp_mp)
    assert np.array_equal(rows[:, 1], want.log_ratio)
    assert np.array_equal(rows[:, 2], want.train.count.astype(np.float64))
    assert got["t_max"] == 10.0 + world - 1


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`bench.py --gpus 2` started plainly: it must launch two ranks itself (torch.distributed.run
    on 127.0.0.1), which here only rendezvous over gloo, shard the rows and reduce a number."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--dry-run-ranks"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["max_over_ranks"] == 2.0 and line["scaling"] == "weak"
    assert line["rows_per_rank"] == inputs.WORKLOADS["c2_bf16_fwdbwd"].T
