// Scalar steps of the iteration that the paper runs on the host (Algorithm 2, steps (d), (e), (g)),
// kept on the device here: one thread executes them after the reductions.  Shared by all kernel
// families so that every path takes the gate / stop decisions with the same arithmetic.
#pragma once
#include "nlr_common.cuh"

namespace gemnlr {

// After the vector pass (and, unless mode == 1, the Theta reduction).
// Finishes the previous iteration: rho = ||q|| / sqrt(n), stop = gate && delta_hat < eps_c &&
// rho < eps_c && t + 1 >= T_min, history record.  mode 0: start of an iteration (records the
// objective the iteration starts from), 1: tail after the U buffer was rescaled (multiplier
// reset to 1), 2: objective evaluation only.
__device__ __forceinline__ void fin1_scalars(Ctl* ctl, double qq, double yq, double t2, int64_t n,
                                             double gamma, double eps_c, int T_min,
                                             gem_nlr_iter_info* hist, int mode, bool combined = false)
{
    ctl->qq = qq;
    ctl->yq = yq;
    if (mode != 1) ctl->theta2 = t2;
    // row-sharded run: these are one rank's sums; they stay parked until the exchange has combined all ranks'
    if (ctl->shard_world > 1 && !combined) return;
    if (ctl->tail_pending) {
        gem_nlr_iter_info rec = ctl->last;
        rec.rho = sqrt(qq / (double)n);
        rec.stop = (rec.dual_applied && rec.delta_hat < eps_c && rec.rho < eps_c &&
                    rec.t + 1 >= T_min) ? 1 : 0;
        ctl->last = rec;
        if (ctl->hist_cap > 0 && rec.t < ctl->hist_cap) {
            hist[rec.t] = rec;
            ctl->hist_len = rec.t + 1;
        }
        ctl->tail_pending = 0;
        ctl->dual_pending = 0;
        if (rec.stop) { ctl->stopped = 1; ctl->status = GEM_NLR_CONVERGED; }
    }
    if (mode != 1) {
        const double f = -t2 + yq + 0.5 * gamma * qq;
        if (mode == 0) ctl->fhat_cur = f;
        if (mode == 2 || ctl->stopped) ctl->f_final = f;
    } else {
        ctl->c_f = 1.0f;
    }
}

// After the fused second product: nu = sqrt(a); breakdown if nu <= 1e-20; c_f = FP32(sqrt(K)/nu);
// Delta = max{c^2 a + b - 2 c h, 0}; delta_hat = sqrt(Delta)/sqrt(K); gate = Delta < eps_d^2 K.
// Returns false on breakdown / non-finite statistics; *c_out = FP64(c_f) otherwise.
__device__ __forceinline__ bool fin2_scalars(Ctl* ctl, double a, double b, double h, int K,
                                             double eps_d, double* c_out, bool combined = false)
{
    if (ctl->shard_world > 1 && !combined) {
        // row-sharded run: park this rank's sums; with c = 1 the caller stores its plain column sums in p
        ctl->sa = a; ctl->sb = b; ctl->sh = h;
        *c_out = 1.0;
        return true;
    }
    gem_nlr_iter_info rec;
    rec.t = ctl->t;
    rec.dual_applied = 0;
    rec.stop = 0;
    rec.status = GEM_NLR_OK;
    rec.a = a; rec.b = b; rec.h = h;
    rec.c = 0.0; rec.delta_hat = 0.0; rec.rho = 0.0;
    rec.fhat = ctl->fhat_cur;
    bool ok = true;
    double c = 1.0;
    if (!isfinite(a) || !isfinite(b) || !isfinite(h)) {
        rec.status = GEM_NLR_E_NONFINITE; ok = false;
    } else {
        const double nu = sqrt(a);
        if (nu <= 1e-20) {
            rec.status = GEM_NLR_E_BREAKDOWN; ok = false;
        } else {
            const float cf = (float)(sqrt((double)K) / nu);
            c = (double)cf;
            double Delta = c * c * a + b - 2.0 * c * h;
            if (Delta < 0.0) Delta = 0.0;
            rec.c = c;
            rec.delta_hat = sqrt(Delta) / sqrt((double)K);
            rec.dual_applied = (Delta < eps_d * eps_d * (double)K) ? 1 : 0;
            ctl->c_f = cf;
            ctl->dual_pending = rec.dual_applied;
            ctl->tail_pending = 1;
            ctl->t = rec.t + 1;
        }
    }
    if (!ok) {
        ctl->c_f = 1.0f;          // the buffer holds W as the paper's loop leaves it
        ctl->stopped = 1;
        ctl->status = rec.status;
        ctl->dual_pending = 0;
        ctl->tail_pending = 0;
    }
    ctl->last = rec;
    *c_out = c;
    return ok;
}

}  // namespace gemnlr
