"""Stored trajectory of the tiny benchmark shape (tests/golden/tiny_trajectory.txt, written by
tests/golden/make_golden.py from the CPU oracle alone): the oracle must still reproduce it, and the GPU
path must match these stored values, which only the oracle can write (a guard against drift of either
side, not an independent pin of the oracle)."""
import hashlib
import importlib.util
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLD = os.path.join(HERE, "golden", "tiny_trajectory.txt")


def _load():
    norm, rows, digest = None, [], None
    for line in open(GOLD):
        if line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "spectral_norm":
            norm = float(tok[1])
        elif tok[0] == "labels_sha256":
            digest = tok[1]
        else:
            rows.append((int(tok[0]), int(tok[1]), *map(float, tok[2:])))
    return norm, rows, digest


def test_oracle_reproduces_the_stored_trajectory():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    norm, rows, digest = _load()
    a_norm, now, dig_now = mg.trajectory()
    assert abs(a_norm - norm) <= 1e-12 * norm
    assert len(now) == len(rows) == mg.ITERS
    for r_old, r_new in zip(rows, now):
        assert r_old[:2] == r_new[:2]
        for x, y in zip(r_old[2:], r_new[2:]):
            assert abs(x - y) <= 1e-9 * max(abs(x), 1e-6), (r_old, r_new)    # thread count may differ: FP64 sum order
    assert dig_now == digest


@pytest.mark.gpu
def test_gpu_matches_the_stored_trajectory():
    import torch
    import synth
    import paper_2609_36074_b200 as gem
    norm, rows, digest = _load()
    spec = synth.config(1)
    hp = synth.default_hparams(spec.K)
    X, _, _ = synth.make_mixture(spec)
    U0 = synth.make_u0(spec.n, spec.K, spec.K)
    T = len(rows)
    s = gem.GemNlr(torch.from_numpy(X).cuda(), torch.from_numpy(U0).cuda(), spec.K, alpha=hp["alpha"], beta=hp["beta"],
                   eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=T, T_min=T, history=1)
    a = s.spectral_norm()
    assert abs(a - norm) <= 1e-5 * norm and a <= norm * (1 + 1e-9)
    rc, info, iters = s.run()
    assert rc == gem.ITER_CAP and iters == T
    hist = s.history(T)
    for h, r in zip(hist, rows):
        t, dual, a_, b_, h_, c_, dh, rho, fh = r
        assert h["t"] == t and h["dual_applied"] == dual
        # free-running FP32 trajectory on the library's own X-hat: looser than the teacher-forced bounds
        for got, want, tol in ((h["a"], a_, 2e-4), (h["b"], b_, 2e-4), (h["h"], h_, 2e-4), (h["c"], c_, 1e-4),
                               (h["rho"], rho, 2e-4)):
            assert abs(got - want) <= tol * abs(want), (t, got, want)
        assert abs(h["delta_hat"] - dh) <= 1e-4
        assert abs(h["fhat"] - fh) <= 2e-4 * max(abs(fh), spec.K / 100)
    lab = s.labels().cpu().numpy().astype(np.int32)
    assert hashlib.sha256(lab.tobytes()).hexdigest() == digest
    s.destroy()
