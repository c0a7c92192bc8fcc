"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks on 127.0.0.1 shard the KV heads, pass the start
barrier and agree on the maximum / sum over ranks."""
import os
import subprocess
import sys

import pytest

from paper_2604_03260_b200 import multi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
from paper_2604_03260_b200 import multi
rank, world, local = multi.env_world()
dist = multi.init("gloo")
multi.barrier(dist)
shard = multi.head_shard(rank, world, 32, 8)
mx = multi.max_over_ranks(10.0 + rank, dist)
sm = multi.sum_over_ranks(float(shard[1] - shard[0]), dist)
print(json.dumps(dict(rank=rank, world=world, shard=shard, mx=mx, sm=sm)), flush=True)
dist.destroy_process_group()
"""


def test_head_shards_partition_the_heads():
    for Hq, Hkv in ((32, 8), (12, 12), (16, 8), (8, 1)):
        for world in (1, 2, 3, 4, 8, 16):
            kv, qh = [], []
            for r in range(world):
                lo, hi, qlo, qhi = multi.head_shard(r, world, Hq, Hkv)
                kv += list(range(lo, hi)); qh += list(range(qlo, qhi))
                assert qlo == lo * (Hq // Hkv) and qhi == hi * (Hq // Hkv)
            assert kv == list(range(Hkv)) and qh == list(range(Hq))
    sizes = [multi.head_shard(r, 3, 32, 8)[1] - multi.head_shard(r, 3, 32, 8)[0] for r in range(3)]
    assert sizes == [3, 3, 2]
    with pytest.raises(ValueError):
        multi.head_shard(0, 2, 10, 4)


def test_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    import socket
    with socket.socket() as sk:                      # a port that is free right now
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert [o["shard"] for o in outs] == [[0, 4, 0, 16], [4, 8, 16, 32]]
    assert all(o["mx"] == 11.0 and o["sm"] == 8.0 and o["world"] == 2 for o in outs)
