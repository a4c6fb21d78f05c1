"""gem_nlr_column_sums_static -- the entry point for callers that cannot allocate device memory
when they call (all device memory handed out at start-up, or an allocation's synchronization not
acceptable): it must give the same column sums p = U^T 1 as the regular, workspace-based path.

This file is named so that pytest collects it last: a run that stops at the first failure has
then already run every other test.  It passes alone in a fresh process as well as after the
other tests, because the entry point looks up its built-in scratch array on its first call."""
import numpy as np
import pytest
import torch

import synth
import paper_2609_36074_b200 as gem

pytestmark = pytest.mark.gpu


def _reference_p(U_host: np.ndarray) -> np.ndarray:
    """p from the existing entry points: a fresh handle computes p = U^T 1 for the loaded factor
    when the objective is first evaluated; gem_nlr_buffer exposes it."""
    n, r = U_host.shape
    Xd = torch.zeros((n, 4), device="cuda")
    Ud = torch.from_numpy(U_host).cuda()
    s = gem.GemNlr(Xd, Ud, min(r, 4), precision=2)
    s.set_normalized(1.0)
    s.objective()
    p = s.buffer(1, r).cpu().numpy().copy()
    s.destroy()
    return p


def test_column_sums_static_matches_workspace_path_twice_in_a_row():
    n, r = 70001, 24                      # many blocks, ragged last block, r not a multiple of 32
    U1 = synth.make_u0(n, r, 4, seed=5)
    U2 = (3.0 * synth.make_u0(n, r, 4, seed=6)).astype(np.float32)
    out = torch.full((r,), float("nan"), device="cuda")
    # two calls in a row on different factors: the second must not see the first one's partial sums
    for U in (U1, U2):
        Ud = torch.from_numpy(U).cuda()
        rc, p = gem.column_sums_static(Ud, out=out)
        assert rc == gem.OK
        torch.cuda.synchronize()
        got = p.cpu().numpy()
        ref = _reference_p(U)
        np.testing.assert_allclose(got, ref, rtol=1e-6, atol=0)
        np.testing.assert_allclose(got, U.astype(np.float64).sum(0), rtol=1e-6, atol=0)
    # a small problem right after a large one: fewer blocks than the scratch still holds records for
    Us = synth.make_u0(37, 5, 2, seed=7)
    rc, p = gem.column_sums_static(torch.from_numpy(Us).cuda())
    torch.cuda.synchronize()
    assert rc == gem.OK
    np.testing.assert_allclose(p.cpu().numpy(), _reference_p(Us), rtol=1e-6, atol=0)


def test_column_sums_static_refuses_sizes_beyond_its_scratch():
    r = gem.STATIC_MAX_R + 1
    U = torch.ones((64, r), device="cuda")
    out = torch.full((r,), -1.0, device="cuda")
    rc, _ = gem.column_sums_static(U, out=out)
    torch.cuda.synchronize()
    assert rc == gem.E_TOO_LARGE
    assert (out == -1.0).all()            # nothing was launched
    rc, p = gem.column_sums_static(torch.ones((64, gem.STATIC_MAX_R), device="cuda"))
    torch.cuda.synchronize()
    assert rc == gem.OK and (p == 64.0).all()
