"""Row-sharded iteration on one GPU: the ranks are handles on disjoint row blocks driven by one host thread each
(paper_2609_36074_b200.sharding.ThreadRanks); the threads meet only at host barriers with no kernel in flight, so
no kernel waits on another.  The sharded result must equal the single-handle result up to the rounding of the
per-rank partial sums, and the oracle within the usual tolerances."""
import threading

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2609_36074_b200 as gem
from paper_2609_36074_b200 import sharding
from gpu_helpers import u_err

pytestmark = pytest.mark.gpu


def _run_sharded(X, U0, K, hp, T, world, precision=-1):
    n = X.shape[0]
    ranges = sharding.row_ranges(n, world)
    ranks = sharding.ThreadRanks(world)
    out = [None] * world
    errs = []

    def work(g):
        try:
            lo, hi = ranges[g]
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                Xd = torch.from_numpy(X[lo:hi].copy()).cuda()
                Ud = torch.from_numpy(U0[lo:hi].copy()).cuda()
                st.synchronize()
                s = gem.GemNlr(Xd, Ud, K, stream=st, alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"],
                               eps_c=hp["eps_c"], T=T, T_min=hp["T_min"], history=1, precision=precision)
                sharding.attach(s, ranks.member(g), n)
                a = s.spectral_norm()
                f0 = s.objective()
                rc, info, iters = s.run()
                lab = s.labels()
                st.synchronize()
                out[g] = dict(a=a, f0=f0, rc=rc, info=info, iters=iters, U=Ud.cpu().numpy(), lab=lab.cpu().numpy(),
                              yt=s.get_state()[0].cpu().numpy(), hist=s.history(T), path=s.path(),
                              Xhat=Xd.cpu().numpy())
                s.destroy()
        except Exception as e:          # a dead rank must not leave the others at the barrier
            errs.append(e)
            ranks.barrier.abort()

    threads = [threading.Thread(target=work, args=(g,)) for g in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errs, errs
    return out


# (n, d, K, world): the general-shape kernels, the warp-level tensor-core family, the tcgen05 fp16-split pair (every
# shard keeps n >= 4096 rows), the TMA-staged FFMA family; two and three ranks, uneven row blocks
@pytest.mark.parametrize("n,d,K,world", [(6001, 16, 4, 2), (9001, 128, 16, 2), (12400, 64, 100, 3), (10001, 32, 8, 2), (8801, 288, 300, 2)])
def test_sharded_run_matches_single_gpu_and_oracle(n, d, K, world):
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 0)
    X, _, _ = synth.make_mixture(spec)
    U0 = synth.make_u0(n, K, K)
    hp = dict(synth.default_hparams(K), eps_d=0.2, T_min=4)
    T = 14
    res = _run_sharded(X, U0, K, hp, T, world)

    # single handle on all rows
    Xd, Ud = torch.from_numpy(X.copy()).cuda(), torch.from_numpy(U0.copy()).cuda()
    s = gem.GemNlr(Xd, Ud, K, alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=T,
                   T_min=hp["T_min"], history=1)
    a1 = s.spectral_norm()
    f01 = s.objective()
    rc1, info1, iters1 = s.run()
    U1 = Ud.cpu().numpy()
    lab1 = s.labels().cpu().numpy()
    hist1 = s.history(T)
    s.destroy()

    # replicated scalars are bit-identical on all ranks
    for g in range(1, world):
        assert res[g]["a"] == res[0]["a"] and res[g]["info"] == res[0]["info"] and res[g]["f0"] == res[0]["f0"]
        assert res[g]["hist"] == res[0]["hist"]
    assert abs(res[0]["a"] - a1) <= 1e-9 * a1
    assert abs(res[0]["f0"] - f01) <= 1e-6 * max(abs(f01), K / 100)
    assert res[0]["rc"] == rc1 and res[0]["iters"] == iters1 == T
    Us = np.concatenate([r["U"] for r in res])
    assert u_err(Us, U1) <= 2e-5, u_err(Us, U1)
    assert [h["dual_applied"] for h in res[0]["hist"]] == [h["dual_applied"] for h in hist1]
    assert sum(h["dual_applied"] for h in hist1) > 0          # the gated dual step took part
    for key in ("rho", "delta_hat", "fhat"):
        assert abs(res[0]["info"][key] - info1[key]) <= 1e-5 * max(abs(info1[key]), 1e-3), key
    labs = np.concatenate([r["lab"] for r in res])
    assert np.mean(labs != lab1) <= 1e-3

    # and the oracle, on the sharded run's own X-hat
    Xhat = np.concatenate([r["Xhat"] for r in res])
    Uo, yto, infoo, _, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], T, hp["T_min"])
    assert u_err(Us, Uo) <= 1e-4
    yts = np.concatenate([r["yt"] for r in res])
    assert float(np.abs(yts - yto).max()) <= 1e-4 * float(np.abs(yto).max()) + 1e-9
    assert abs(res[0]["info"]["rho"] - infoo["rho"]) <= 1e-4 * infoo["rho"]


def test_single_gpu_calls_are_refused_on_a_sharded_handle():
    n, d, K = 5000, 16, 4
    X = np.random.default_rng(0).standard_normal((n, d)).astype(np.float32)
    U0 = synth.make_u0(n, K, K)
    # a handle that holds half of the rows of a two-rank problem (its peer never runs: nothing is exchanged here)
    ranks = sharding.ThreadRanks(2)
    s = gem.GemNlr(torch.from_numpy(X).cuda(), torch.from_numpy(U0).cuda(), K)
    sharding.attach(s, ranks.member(0), 2 * n)
    s.set_normalized(1.0)
    assert s.init_range() == gem.E_INVALID
    assert s.labels_spectral()[0] == gem.E_INVALID
    s.destroy()
    # one rank: attaching changes nothing
    s = gem.GemNlr(torch.from_numpy(X).cuda(), torch.from_numpy(U0).cuda(), K)
    sharding.attach(s, sharding.ThreadRanks(1).member(0), n)
    s.spectral_norm()
    rc, info = s.step()
    assert rc == gem.OK and s.init_range() == gem.OK
    s.destroy()
