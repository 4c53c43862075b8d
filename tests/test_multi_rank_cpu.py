"""World-size-2 check (gloo, CPU) of the rank partition used for N > 1: the
shards cover every (batch, KV head) unit exactly once, need no exchange, and
their results gathered over ranks equal the unsharded result.  The per-shard
compute stands in with the CPU oracle (no GPU here); on GPUs each rank calls
the CUDA library on the same slices."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2604_18616_b200 import inputs, shard


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_path):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.small_variant(inputs.get("c3_gqa_prefill"), B=3, H=8, Hkv=2, Sq=40, Sk=56, D=16)
        q, k, v = inputs.make_inputs(w)                     # every rank derives the same seeded problem
        qu, ku, vu, (lo, hi) = shard.shard_qkv(q, k, v, world, rank)
        o, lse = oracle.attn_fwd(qu.contiguous(), ku.contiguous(), vu.contiguous(), w.causal, w.scale)
        # timing reduction used by the benchmark: max over ranks
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == world
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, o, lse))
        if rank == 0:
            units = sorted((g[0], g[1]) for g in gathered)
            assert units[0][0] == 0 and units[-1][1] == w.B * w.Hkv
            assert all(units[i][1] == units[i + 1][0] for i in range(len(units) - 1))
            o_all = np.concatenate([g[2] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
            l_all = np.concatenate([g[3] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
            o_ref, l_ref = oracle.attn_fwd(q, k, v, w.causal, w.scale)
            assert np.array_equal(o_all.reshape(o_ref.shape), o_ref)
            assert np.array_equal(l_all.reshape(l_ref.shape), l_ref)
            open(out_path, "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_unit_ranges_cover_everything_once():
    for n in (1, 2, 7, 8, 64):
        for world in (1, 2, 3, 8):
            spans = [shard.unit_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.unit_range(4, 2, 2)


def test_two_ranks_gloo(tmp_path):
    oracle.build()
    out = tmp_path / "ok.txt"
    mp.spawn(_worker, args=(2, _free_port(), str(out)), nprocs=2, join=True)
    assert out.read_text() == "ok"


@pytest.mark.parametrize("scaling", ["weak", "strong"])
def test_bench_gpus_2_starts_two_ranks(scaling):
    """`bench.py --gpus 2` with no torchrun environment starts the two ranks itself; `--plan-only` stops
    after the rendezvous (gloo here, NCCL on GPUs) and reports which rank would run what."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plan-only", "--scaling", scaling,
                        "--workload", "c3_gqa_prefill"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["scaling"] == scaling
    plan = sorted(line["plan"], key=lambda p: p["rank"])
    assert [p["rank"] for p in plan] == [0, 1] and [p["local_rank"] for p in plan] == [0, 1]
    if scaling == "weak":          # an independent batch per rank
        assert plan[0]["seed"] != plan[1]["seed"] and plan[0]["units"] == plan[1]["units"] == [0, 16]
    else:                          # the (batch, KV head) units of one batch, split without overlap
        assert plan[0]["seed"] == plan[1]["seed"]
        assert plan[0]["units"] == [0, 8] and plan[1]["units"] == [8, 16]
