"""Host side of the row-sharded run on two gloo ranks on the CPU: row blocks, the all-gather callback (records back
to back in rank order) and the rank-ordered host sum, exercised through the same callback objects the library
calls.  No kernel runs here."""
import json
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import ctypes as C, json, os, sys
    sys.path.insert(0, os.environ["REPO_ROOT"])
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2609_36074_b200 import sharding
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ex = sharding.TorchDistExchange()
    xcount = 7
    xbuf = torch.zeros((world + 1) * xcount, dtype=torch.float64)
    ex.bind(xbuf, None)
    count = 5                                         # a record shorter than the area it was sized for
    xbuf[:count] = torch.arange(count, dtype=torch.float64) + 100.0 * rank
    base = xbuf.data_ptr()
    # call through the C function pointers, as the library does
    rc = ex.gather_c(None, base, base + 8 * xcount, 8 * count, None)
    recv = xbuf[xcount: xcount + world * count].tolist()
    bad = ex.gather_c(None, base + 8, base + 8 * xcount, 8 * count, None)     # foreign pointer: refused, no exception
    # rank-ordered host sum: (1e16 + 1) - 1e16 differs from 1e16 + (1 - 1e16) in FP64
    vec = (C.c_double * 3)(*([1e16, 3.0, 0.5] if rank == 0 else [1.0, 4.0, 0.25]))
    rc2 = ex.host_sum_c(None, vec, 3)
    print("RESULT " + json.dumps(dict(rank=rank, rc=rc, bad=bad, recv=recv, rc2=rc2, vec=list(vec))), flush=True)
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_exchange_callbacks_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    res = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        res.append(json.loads([l for l in out.splitlines() if l.startswith("RESULT ")][0][7:]))
    res.sort(key=lambda d: d["rank"])
    want = [0.0, 1.0, 2.0, 3.0, 4.0, 100.0, 101.0, 102.0, 103.0, 104.0]
    for d in res:
        assert d["rc"] == 0 and d["rc2"] == 0 and d["bad"] == 1
        assert d["recv"] == want                                  # both ranks: rank 0's record, then rank 1's
        assert d["vec"] == [1e16 + 1.0, 7.0, 0.75]                # rank 0 + rank 1, in that order, on both ranks


def test_row_ranges_and_ordered_sum():
    from paper_2609_36074_b200 import sharding
    assert sharding.row_ranges(10, 3) == [(0, 4), (4, 7), (7, 10)]
    assert sharding.row_ranges(7, 7) == [(i, i + 1) for i in range(7)]
    r = sharding.row_ranges(100_000_001, 8)
    assert r[0][0] == 0 and r[-1][1] == 100_000_001 and all(a[1] == b[0] for a, b in zip(r, r[1:]))
    assert max(hi - lo for lo, hi in r) - min(hi - lo for lo, hi in r) == 1
    parts = [np.array([1e16]), np.array([1.0]), np.array([-1e16])]
    assert sharding.ordered_sum(parts)[0] == (1e16 + 1.0) - 1e16   # left to right, not pairwise or sorted


def test_thread_ranks_gather_on_host_memory():
    """The in-process stand-in for the ranks (used by the single-GPU tests) obeys the same contract."""
    import threading
    import torch
    from paper_2609_36074_b200 import sharding
    world, xcount, count = 3, 6, 4
    ranks = sharding.ThreadRanks(world)
    exs = [ranks.member(g) for g in range(world)]
    bufs = [torch.zeros((world + 1) * xcount, dtype=torch.float64) for _ in range(world)]
    for g in range(world):
        exs[g].bind(bufs[g], None)
        bufs[g][:count] = torch.arange(count, dtype=torch.float64) + 10.0 * g
    sums = [None] * world

    def work(g):
        base = bufs[g].data_ptr()
        assert exs[g].gather_c(None, base, base + 8 * xcount, 8 * count, None) == 0
        sums[g] = exs[g].host_sum(np.array([float(g + 1), 1e16 if g == 0 else (1.0 if g == 1 else -1e16)]))

    ts = [threading.Thread(target=work, args=(g,)) for g in range(world)]
    for t in ts:
        t.start()
    for t in ts:
        t.join(timeout=60)
    want = [float(v + 10 * g) for g in range(world) for v in range(count)]
    for g in range(world):
        assert bufs[g][xcount: xcount + world * count].tolist() == want
        assert sums[g].tolist() == [6.0, (1e16 + 1.0) - 1e16]
