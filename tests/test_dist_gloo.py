"""The N>1 plumbing on CPU: two gloo ranks, max-over-ranks timing, row sharding."""
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["RG_ROOT"])
import numpy as np
from paper_2609_11356_b200 import dist
rank, local_rank, world = dist.init("gloo")
dist.barrier()
mx = dist.max_over_ranks(10.0 + rank)
sm = dist.sum_over_ranks(1.0 + rank)
lo, hi = dist.shard_rows(11, rank, world)
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "max": mx, "sum": sm, "lo": lo, "hi": hi}))
dist.finalize()
"""


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def test_two_gloo_ranks_agree_on_max_and_cover_all_rows():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), RG_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0
        outs.append(eval(out.strip().splitlines()[-1].replace("true", "True")))
    assert all(o["max"] == 11.0 and o["sum"] == 3.0 and o["world"] == 2 for o in outs)
    spans = sorted((o["lo"], o["hi"]) for o in outs)
    assert spans == [(0, 6), (6, 11)]


def test_shard_rows_partitions_exactly():
    from paper_2609_11356_b200 import dist
    for total in (0, 1, 7, 64, 65536):
        for world in (1, 2, 3, 8):
            spans = [dist.shard_rows(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
