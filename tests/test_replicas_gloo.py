"""The multi-GPU form of the path on CPU: two gloo ranks, each an independent replica.

Each rank drives its own bookkeeping-only library context and its own checker through the tiny
workload's script (tables must match id for id on every rank: nothing of one replica reaches the
other), then the ranks aggregate the measurement the way bench.py does: the slowest replica defines
the time, the units add up.  Also checked: the replica seeds differ, and the reference arm of
bench.py stays silent on ranks other than 0.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B, replicas, workloads as wl

g = replicas.Group("gloo")
rank, world, _ = replicas.env()
assert g.active and g.world == 2
w = wl.tiny()
sh = w.shape
lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads, head_dim=sh.head_dim,
               block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks, max_blocks_per_req=32, host_pool_bytes=1 << 30,
               initial_free_order=w.free_order, flags=B.PS_FLAG_BOOKKEEPING_ONLY)
orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size, sh.num_gpu_blocks, w.free_order)
for r, n in wl.build_order_round_robin(w):
    assert lib.kv_alloc(r, n) == orc.kv_alloc(r, n) == 0
victims = w.victims if rank == 0 else w.victims[:2]          # the replicas need not do the same thing
for r in victims:
    assert lib.swap_out(r) == orc.swap_out(r) == 0
assert lib.sync() == 0
orc.reap()
g.barrier()
for r in victims:
    assert lib.swap_in_begin(r) == orc.swap_in_begin(r) == 0
reqs = list(range(len(w.ctx_lens)))
rc, mask, st = lib.step(None, None, reqs, -1)
plan, omask, _ = orc.step(-1, reqs)
assert rc == 0 and mask == omask
for r in reqs:
    assert lib.block_table(r) == orc.block_table(r)
units = st["h2d_bytes"]
ms_local = 10.0 * (rank + 1)                                 # rank 1 is the slow replica
rate, ms = replicas.whole_job_rate(g, units, ms_local)
mx = g.max_over_ranks([ms_local, -ms_local])
sm = g.sum_over_ranks([units])
print(json.dumps({{"rank": rank, "units": units, "rate": rate, "ms": ms, "max": mx, "sum": sm,
                  "seed": replicas.replica_seed(w.seed, rank)}}))
g.close()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_replicas_are_independent_and_aggregate_like_the_bench(tmp_path):
    from paper_2512_12928_b200 import build as ps_build
    ps_build.build()
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            o, e = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    units = [d["units"] for d in outs]
    assert units[0] > units[1] > 0                           # rank 0 reloaded four requests, rank 1 two
    for d in outs:
        assert d["ms"] == 20.0                               # the slowest replica defines the step
        assert d["max"] == [20.0, -10.0]
        assert d["sum"] == [float(sum(units))]
        assert d["rate"] == pytest.approx(sum(units) / 20e-3)
    assert outs[0]["seed"] != outs[1]["seed"]


SPAWNED = r"""
import json, os, sys
sys.path.insert(0, {root!r})
from paper_2512_12928_b200 import binding as B, replicas
g = replicas.Group("gloo")
rank, world, local = replicas.env()
lib = B.KVSwap(num_layers=2, num_kv_heads=2, num_q_heads=4, head_dim=64, block_size=16, num_gpu_blocks=32,
               max_blocks_per_req=8, host_pool_bytes=1 << 20, flags=B.PS_FLAG_BOOKKEEPING_ONLY)
assert lib.kv_alloc(rank, 40 * (rank + 1)) == 0
blocks = len(lib.block_table(rank)[0])
(total,) = g.sum_over_ranks([blocks])
open(os.path.join({out!r}, f"rank{{rank}}.json"), "w").write(json.dumps(
    {{"rank": rank, "world": world, "local": local, "addr": os.environ["MASTER_ADDR"], "total": total}}))
g.close()
"""


def test_spawn_starts_one_replica_per_rank_with_a_launcher_environment(tmp_path):
    """What `bench.py --gpus N` does without a launcher: N processes with RANK / LOCAL_RANK / WORLD_SIZE and a
    rendezvous on 127.0.0.1, here with bookkeeping-only contexts over gloo."""
    from paper_2512_12928_b200 import build as ps_build, replicas
    ps_build.build()
    script = tmp_path / "spawned.py"
    script.write_text(SPAWNED.format(root=ROOT, out=str(tmp_path)))
    rcs = replicas.spawn([sys.executable, str(script)], 2)
    assert rcs == [0, 0]
    outs = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in range(2)]
    assert [d["rank"] for d in outs] == [0, 1] and [d["local"] for d in outs] == [0, 1]
    assert all(d["world"] == 2 and d["addr"] == "127.0.0.1" for d in outs)
    assert all(d["total"] == 3.0 + 5.0 for d in outs)          # ceil(40 / 16) + ceil(80 / 16) blocks


def test_cpulist_parsing_and_missing_numa_information():
    from paper_2512_12928_b200 import replicas
    assert replicas.parse_cpulist("0-3,8,10-11\n") == [0, 1, 2, 3, 8, 10, 11]
    assert replicas.parse_cpulist("") == []
    assert replicas.numa_cpus_of_gpu(0, sysfs="/nonexistent") is None     # no such box: nothing is bound


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=240)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_single_process_group_is_a_no_op():
    from paper_2512_12928_b200 import replicas
    env = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        g = replicas.Group("gloo")
        assert not g.active
        g.barrier()
        assert g.max_over_ranks([3.0, 1.5]) == [3.0, 1.5] and g.sum_over_ranks([2]) == [2.0]
        assert replicas.whole_job_rate(g, 100.0, 50.0) == (2000.0, 50.0)
        g.close()
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v
