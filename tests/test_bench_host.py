"""Host-side logic of bench.py: the roofline byte model, mask recipes, and the N>1 aggregation
(replicas only: max over ranks of the device time, tokens summed over ranks) under gloo."""
import os
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402
import first_inputs as fi  # noqa: E402


def test_byte_model_matches_hand_count():
    s = fi.LLAMA_8B
    mask = np.ones((2, s.n_layers), np.uint8)
    mask[:, 5] = 0          # a layer nobody keeps: its weights are not read
    mask[1, 7] = 0          # one row skips layer 7: only its KV drops out
    lens = np.array([100, 200])
    bm = bench.byte_model(s, mask, lens)
    w_layer = 2 * ((4096 + 2 * 1024) * 4096 + 4096 * 4096 + 3 * 14336 * 4096)
    assert w_layer == 436207616
    kv_tok = 2 * 1024 * 2
    kv = kv_tok * (101 * 31 + 201 * 30)
    assert bm["weights"] == 31 * w_layer and bm["kv"] == kv and bm["strict"] == 31 * w_layer + kv
    assert bm["lm_head"] == 128256 * 4096 * 2
    assert bm["full"] == bm["strict"] + bm["lm_head"] + 2 * 4096 * 2 + (31 + 30) * kv_tok + 2 * 128256 * 4


def test_mask_recipes_have_the_stated_structure():
    m = fi.mask_skip_fraction(32, 32, 0.1, 0.4, 1)
    assert m[:, 0].all() and m[:, -1].all()
    skipped = 32 - m.sum(1)
    assert skipped.min() >= 3 and skipped.max() <= 13
    a = fi.mask_aligned(8, 32, 0.25)
    assert (a == a[0]).all() and (32 - a[0].sum()) == 8 and a[0, 0] and a[0, -1]
    i = fi.mask_independent(8, 32, 0.25, 3)
    assert ((32 - i.sum(1)) == 8).all() and not (i == i[0]).all()
    u = fi.mask_unified(4, 32, 4)     # layers 3, 7, ..., 27 (31 is the last layer and stays)
    assert (u == u[0]).all() and [l for l in range(32) if not u[0, l]] == list(range(3, 31, 4))
    assert fi.mask_unified(2, 32, 0).all()
    r = fi.mask_random_shared(8, 32, 0.25, 5)
    assert (r == r[0]).all() and (32 - r[0].sum()) == 8 and r[0, 0] and r[0, -1]
    assert not (r[0] == fi.mask_random_shared(8, 32, 0.25, 6)[0]).all()
    b = fi.mask_bernoulli(256, 32, 0.7, 2)
    assert b[:, 0].all() and b[:, -1].all() and 0.6 < b[:, 1:-1].mean() < 0.8


def _rank_main(rank, world, port, q):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 100.0 + 25.0 * rank          # rank 1 is the slow replica
    got = bench.max_over_ranks(ms, dist, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, got))


def test_replica_aggregation_over_two_gloo_ranks():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == {0: 125.0, 1: 125.0}       # both ranks agree on the slowest time
    assert bench.job_tokens_per_s(2, 32, 10, 125.0) == 2 * 32 * 10 / 0.125
    assert bench.max_over_ranks(7.5, None, None) == 7.5


_STUB = '''
import json, os, sys
sys.path.insert(0, {root!r})
import torch
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["FIRST_BENCH_BACKEND"] == "gloo" and os.environ["LOCAL_RANK"] == "0"
dist.init_process_group("gloo")                      # MASTER_ADDR / MASTER_PORT from the spawner
ms = bench.max_over_ranks(100.0 + 25.0 * rank, dist, torch.device("cpu"))
dist.barrier()
rec = dict(rank=rank, world=world, gpu=os.environ["CUDA_VISIBLE_DEVICES"], ms=ms, argv=sys.argv[1:],
           addr=os.environ["MASTER_ADDR"])
open(os.path.join({out!r}, f"rank{{rank}}.json"), "w").write(json.dumps(rec))
if rank == 0:
    print(json.dumps(dict(n_gpus=world, value=bench.job_tokens_per_s(world, 32, 10, ms))))
dist.destroy_process_group()
sys.exit(3 if (rank == 1 and "--fail" in sys.argv) else 0)
'''


def test_gpus_n_starts_n_replicas_one_process_per_gpu(tmp_path, capfd):
    """`bench.py --gpus N` outside torchrun starts the N replicas itself: replica i gets GPU i alone, rank i of N,
    a 127.0.0.1 rendezvous; rank 0's line is passed through; the slowest replica's time is what all agree on.
    A stub stands in for the GPU work (gloo, 2 ranks)."""
    import json
    stub = tmp_path / "stub_worker.py"
    stub.write_text(_STUB.format(root=str(ROOT), out=str(tmp_path)))
    rc = bench.spawn_replicas(2, ["--steps", "10"], script=[str(stub)], timeout=300)
    assert rc == 0
    recs = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in range(2)]
    assert [r["gpu"] for r in recs] == ["0", "1"] and [r["rank"] for r in recs] == [0, 1]
    assert all(r["world"] == 2 and r["ms"] == 125.0 and r["argv"] == ["--steps", "10"] and r["addr"] == "127.0.0.1"
               for r in recs)
    line = json.loads(capfd.readouterr().out.strip().splitlines()[-1])
    assert line == {"n_gpus": 2, "value": 2 * 32 * 10 / 0.125}
    # a failing replica fails the job
    assert bench.spawn_replicas(2, ["--fail"], script=[str(stub)], timeout=300) == 3
