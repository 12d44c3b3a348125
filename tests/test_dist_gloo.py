"""World-size-2 CPU test (gloo) of the multi-GPU plumbing: the path shards by episode with no
exchange step, so the ranks only agree on the slowest rank's time; the shards must cover every
episode exactly once and each shard must be a valid varlen batch of its own."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

from paper_2510_18546_b200 import dist, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_episodes_partitions_and_balances():
    wl = synth.make("concurrent")
    for world in (1, 2, 4, 8):
        shards = dist.shard_episodes(wl.n_q, world)
        flat = sorted(b for s in shards for b in s)
        assert flat == list(range(wl.batch))
        loads = [sum(wl.n_q[b] for b in s) for s in shards]
        assert max(loads) - min(loads) <= max(wl.n_q)
    assert dist.shard_episodes([5, 5, 5], 2) == [[0, 2], [1]]


WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import numpy as np
    from paper_2510_18546_b200 import dist, synth
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group(world, rank, backend="gloo")
    dist.barrier()
    t = dist.max_over_ranks(10.0 + 5.0 * rank)              # the slowest rank decides
    wl = synth.make("concurrent")
    mine = dist.shard_episodes(wl.n_q, world)[rank]
    cs, cq, cn = wl.cu()
    n_q = sum(wl.n_q[b] for b in mine)
    total = dist.max_over_ranks(float(n_q))
    dist.barrier()
    print("RESULT", rank, t, n_q, total, ",".join(map(str, mine)), flush=True)
""")


def test_two_ranks_gloo(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            o, e = p.communicate(timeout=180)
        except subprocess.TimeoutExpired:
            p.kill()
            raise
        assert p.returncode == 0, e[-2000:]
        outs.append([l for l in o.splitlines() if l.startswith("RESULT")][0].split())
    wl = synth.make("concurrent")
    eps = []
    for o in outs:
        assert float(o[2]) == 15.0
        eps += [int(x) for x in o[5].split(",")]
    assert sorted(eps) == list(range(wl.batch))
    assert float(outs[0][4]) == float(outs[1][4]) == max(float(outs[0][3]), float(outs[1][3]))
    assert int(outs[0][3]) + int(outs[1][3]) == int(np.sum(wl.n_q))
