"""The N > 1 protocol of the benchmark (independent replicas, barrier, max over ranks) on two gloo
ranks on the CPU: no kernel runs here, only the host logic the multi-GPU run relies on."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, os.environ["REPO_ROOT"])
    import numpy as np
    import torch.distributed as dist
    import synth
    from paper_2609_36074_b200 import replicas
    rank, world, local = replicas.rank_world_local()
    dist.init_process_group("gloo")
    spec = replicas.replica_spec(synth.config(1), rank)
    X, _, _ = synth.make_mixture(spec)
    replicas.barrier()
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = replicas.max_over_ranks(ms_local)
    replicas.barrier()
    out = dict(rank=rank, world=world, seed=spec.seed, x0=float(X[0, 0]), ms=ms,
               value=replicas.whole_job_rate(world, 4, 25, ms))
    print("RESULT " + json.dumps(out), flush=True)
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_over_gloo(tmp_path):
    import json
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
    assert [d["world"] for d in res] == [2, 2]
    assert res[1]["seed"] == res[0]["seed"] + 1 and res[0]["x0"] != res[1]["x0"]      # independent problems
    assert res[0]["ms"] == res[1]["ms"] == 15.0                                       # slowest rank decides
    assert res[0]["value"] == res[1]["value"] == 2 * 4 * 25 / 15e-3                   # whole-job iterations/s


def test_single_process_is_identity():
    from paper_2609_36074_b200 import replicas
    assert replicas.max_over_ranks(3.25) == 3.25
    replicas.barrier()
    assert replicas.whole_job_rate(1, 5, 100, 25.0) == 20000.0
