"""Writes tests/golden/tiny_trajectory.txt: the per-iteration scalars of the first 25 iterations of the
tiny benchmark shape (config 1: n = 2000, d = 16, K = 4, seed 0) and a digest of the final labels.

The paper prints no worked numerical example, so these stored values are not the paper's: they come
from the CPU oracle alone (this script imports nothing but `oracle` and the input generators) and
serve two purposes: a change of the oracle's arithmetic shows up as a diff of this file, and the GPU
path is compared with stored values that no GPU run can alter (the file was written after the first
kernels existed; it pins the oracle against drift, it is not a pin of the oracle itself).

    python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import synth  # noqa: E402

ITERS = 25
FIELDS = ("a", "b", "h", "c", "delta_hat", "rho", "fhat")


def trajectory():
    spec = synth.config(1)
    hp = synth.default_hparams(spec.K)
    X, _, _ = synth.make_mixture(spec)
    Xhat, a_norm, _ = oracle.normalize(X)
    st = oracle.State(Xhat, synth.make_u0(spec.n, spec.K, spec.K))
    rows = []
    for _ in range(ITERS):
        info = st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
        rows.append((info["t"], info["dual"], *[info[k] for k in FIELDS]))
    lab = oracle.labels(st.U)
    return a_norm, rows, hashlib.sha256(lab.astype(np.int32).tobytes()).hexdigest()


def main():
    a_norm, rows, digest = trajectory()
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_trajectory.txt")
    with open(out, "w") as f:
        f.write("# Algorithm 1 on config 1 (n=2000 d=16 K=4, seed 0), first %d iterations, CPU oracle (FP32 buffers, FP64 sums)\n" % ITERS)
        f.write("# written by tests/golden/make_golden.py; not values printed in the paper (it prints none)\n")
        f.write("spectral_norm %.17g\n" % a_norm)
        f.write("# t dual " + " ".join(FIELDS) + "\n")
        for r in rows:
            f.write("%d %d " % (r[0], r[1]) + " ".join("%.17g" % v for v in r[2:]) + "\n")
        f.write("labels_sha256 %s\n" % digest)
    print("wrote", out)


if __name__ == "__main__":
    main()
