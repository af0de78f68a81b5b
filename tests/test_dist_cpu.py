"""world_size-2 gloo test of the multi-rank host logic (no GPU): the reductions the
benchmark uses for its timings, and the layer sharding rule."""
import os
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
from paper_2510_18269_b200 import dist as sdist
rank, world, local = sdist.init_from_env(2, backend="gloo")
assert world == 2
sdist.barrier()
t = sdist.max_over_ranks(10.0 + rank)          # slowest rank decides the time
u = sdist.sum_over_ranks(100.0 * (rank + 1))   # units add up
b, c = sdist.shard_layers(28, rank, world)
tot = sdist.sum_over_ranks(c)
sdist.finish()
print(f"RESULT {rank} {t} {u} {b} {c} {tot}")
"""


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_rank_reductions_gloo(tmp_path):
    port = free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script), str(ROOT)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    rows = sorted(line.split()[1:] for o, _ in outs for line in o.splitlines() if line.startswith("RESULT"))
    assert [r[0] for r in rows] == ["0", "1"]
    for r in rows:
        assert float(r[1]) == 11.0 and float(r[2]) == 300.0 and float(r[5]) == 28.0
    assert (rows[0][3], rows[0][4], rows[1][3], rows[1][4]) == ("0", "14", "14", "14")


def test_shard_layers_covers_everything():
    from paper_2510_18269_b200 import dist as sdist
    for L in (1, 28, 80):
        for world in (1, 2, 3, 8):
            spans = [sdist.shard_layers(L, r, world) for r in range(world)]
            assert sum(c for _, c in spans) == L
            pos = 0
            for b, c in spans:
                assert b == pos
                pos += c
