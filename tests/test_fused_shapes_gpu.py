"""Parity of the fused tensor-core path (bf16 tensors, d = 64, r <= 64) with the float64 oracle over the
launch geometries it has: fewer slices than SMs (several thread blocks per slice), more slices than SMs,
slice counts that do not divide the SM count, ragged last tiles, key masks, zero and one iteration (no stored
Gibbs kernel), small eps on clustered inputs, and r in each padded width (16, 32, 64)."""
import numpy as np
import pytest
import torch

from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import synth
from lot_testutil import check_slice, gpu_forward, oracle_slice

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def streamed_path():
    """Short sequences take the slice path by default: these cases are about the streamed kernels' geometries."""
    lot.lot_debug_hook(4, 1)
    yield
    lot.lot_debug_hook(4, -1)


CASES = [
    # B, H, n, r, iters, eps, key mask
    (1, 1, 1, 64, 3, 0.1, False),
    (1, 1, 127, 64, 2, 0.1, False),
    (1, 1, 129, 40, 4, 0.1, True),
    (2, 3, 257, 64, 5, 0.1, True),
    (1, 40, 700, 64, 3, 0.1, False),
    (3, 50, 130, 48, 3, 0.2, True),
    (1, 148, 256, 64, 2, 0.1, False),
    (1, 150, 200, 64, 3, 0.1, True),
    (1, 2, 5000, 64, 7, 0.05, False),
    (2, 8, 3000, 33, 6, 0.1, True),
    (1, 16, 2048, 64, 1, 0.1, False),
    (1, 16, 2048, 64, 0, 0.1, False),
    (1, 5, 9000, 64, 4, 0.02, False),
    (1, 300, 129, 64, 3, 0.1, True),
    (4, 4, 1111, 64, 12, 0.3, False),
    (1, 1, 20000, 64, 3, 0.1, False),
    (1, 2, 2048, 64, 6, 0.01, False),
    (1, 7, 1500, 17, 5, 0.1, True),
    (1, 9, 1000, 8, 4, 0.1, False),
    (1, 37, 4096, 64, 3, 0.1, False),
    # many short slices: ten and more (slice, side) pairs per thread block
    (128, 12, 100, 64, 3, 0.1, False),
    (512, 3, 197, 16, 4, 0.1, True),
    (96, 4, 150, 64, 5, 0.01, False),
    # 4096 tiles per side and more: the apply stages run as their own kernels, from the stored Gibbs kernel
    (2, 16, 16384, 64, 3, 0.1, True),
    (1, 33, 16384, 50, 2, 0.1, False),
    # the benchmark shapes of configs 2 and 3 at a training-size batch
    (64, 3, 197, 16, 10, 0.1, False),
    (32, 12, 512, 32, 20, 0.05, True),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "B%d-H%d-n%d-r%d-T%d-eps%g-%s" % (c[:6] + ("mask" if c[6] else "full",)))
def test_fused_path_matches_oracle(case):
    B, H, n, r, iters, eps, masked = case
    x = synth.make(B, H, n, 64, r, seed=1000 + 7 * n + H, dtype=torch.bfloat16, eps=eps, iters=iters,
                   key_len_range=(max(1, n // 2), n) if masked else None, qk="mixture" if eps < 0.03 else "normal")
    res = gpu_forward(x, want_g=True)
    assert res["status"] == 0
    assert np.isfinite(res["out"]).all()
    for (b, h) in sorted({(0, 0), (B // 2, H // 2), (B - 1, H - 1)}):
        ref, g1, g2 = oracle_slice(x, b, h, return_potentials=True)
        check_slice(res["out"][b, h], ref, 2e-2, f"slice {(b, h)}")
        # potentials: stored-kernel passes round the Gibbs kernel to bf16 once (see test_parity_gpu)
        scale = max(1.0, np.abs(g1).max(), np.abs(g2).max())
        assert np.abs(res["g1"][b, h] - g1).max() <= 1e-3 * scale
        assert np.abs(res["g2"][b, h] - g2).max() <= 1e-3 * scale


MIXED = [
    # H, n, iters, scale of q, scale of k: scaled tokens widen the spread of that side's potentials, so that one side of
    # a slice leaves the stored-kernel passes (spread above 64 binades) while the other stays on them
    (4, 3000, 8, 8.0, 1.0),
    (4, 3000, 8, 1.0, 8.0),
    (16, 16384, 10, 8.0, 1.0),
    (3, 2500, 9, 6.0, 6.0),
]


@pytest.mark.parametrize("case", MIXED, ids=lambda c: "H%d-n%d-T%d-q%g-k%g" % c)
def test_fused_path_mixed_pass_kinds(case):
    import dataclasses
    H, n, iters, qs, ks = case
    x = synth.make(1, H, n, 64, 64, seed=11, dtype=torch.bfloat16, eps=0.1, iters=iters)
    x = dataclasses.replace(x, q=(x.q.float() * qs).to(torch.bfloat16), k=(x.k.float() * ks).to(torch.bfloat16))
    res = gpu_forward(x, want_g=True)
    assert res["status"] == 0
    assert np.isfinite(res["out"]).all()
    for h in sorted({0, H - 1}):
        ref, g1, g2 = oracle_slice(x, 0, h, return_potentials=True)
        check_slice(res["out"][0, h], ref, 2e-2, f"head {h}")
        scale = max(1.0, np.abs(g1).max(), np.abs(g2).max())
        assert np.abs(res["g1"][0, h] - g1).max() <= 1e-3 * scale
        assert np.abs(res["g2"][0, h] - g2).max() <= 1e-3 * scale
