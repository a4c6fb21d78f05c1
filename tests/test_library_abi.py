"""Host-only checks of the C ABI: the library loads, exports every declared symbol, and its
closed-form accounting matches the paper's storage formula (no device work)."""
import os
import re

import paper_2609_36074_b200 as gem
from paper_2609_36074_b200.binding import make_params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "gem_nlr.h")).read()
    names = sorted(set(re.findall(r"\b(gem_nlr_[a-z_]+)\s*\(", hdr)))
    assert {"gem_nlr_create", "gem_nlr_spectral_norm", "gem_nlr_step", "gem_nlr_run", "gem_nlr_labels",
            "gem_nlr_destroy"} <= set(names)
    L = gem.lib()
    for name in names:
        assert getattr(L, name) is not None, name


def test_storage_accounting_closed_forms():
    # Eq. "gpu-storage" with 128 x 64 output tiles: 4(nd + nr + dr + 4n + 2r) + 24(N_tile + 1)
    n, d, r = 1_000_000, 128, 16
    P = make_params(n, d, r)
    n_tile = -(-n // 128) * -(-r // 64)
    assert gem.paper_storage_bytes(P) == 4 * (n * d + n * r + d * r + 4 * n + 2 * r) + 24 * (n_tile + 1)
    ws = gem.workspace_bytes(P)
    # beyond X and the single factor the library keeps only O(n) vectors and small partial arrays
    assert 8 * n <= ws <= 8 * n + 64 * 2 ** 20
    assert gem.workspace_bytes(make_params(n, d, r, x_inplace=0)) >= ws + 4 * n * d
    assert gem.workspace_bytes(make_params(0, d, r)) == 0          # invalid
    assert gem.workspace_bytes(make_params(n, d, 4, r=2)) == 0     # r < K


def test_image_workspace_rounds_the_feature_count_up():
    # The tensor-core shapes (r >= 32, n >= 4096) keep fp16 split images of X-hat, row-major and transposed:
    # 8 n d' bytes with d' = d rounded up to a multiple of 32, so d = 50 costs what d = 64 costs there;
    # below n = 4096 and for narrow factors there are no images.
    n, r = 100_000, 60
    base = gem.workspace_bytes(make_params(n, 64, r, precision=2))           # generic only: no images
    w64 = gem.workspace_bytes(make_params(n, 64, r))
    w50 = gem.workspace_bytes(make_params(n, 50, r))
    assert 8 * n * 64 <= w64 - base <= 8 * n * 64 + 64 * 64 * 128 + 2 ** 20
    assert abs(w50 - w64) <= 2 ** 20                                         # Theta and partials sized for d' too
    assert gem.workspace_bytes(make_params(4000, 50, r)) == gem.workspace_bytes(make_params(4000, 50, r, precision=2))
    assert gem.workspace_bytes(make_params(n, 50, 16)) == gem.workspace_bytes(make_params(n, 50, 16, precision=2))
