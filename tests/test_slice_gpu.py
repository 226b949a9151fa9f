"""The slice path (bf16 tensors, d = 64, r <= 64, n <= 512: one thread block per (batch, head) slice, a side's logits
in float32 registers for all iterations) against the float64 oracle: every register shape (pivot widths 16, 32, 64;
one or two 16-row tiles per warp), ragged row counts, key masks (down to one and to no valid key), zero and many
iterations, clustered inputs at small eps (column sums outside float32's range take the recomputation relative to the
column maximum), more slices than SMs.  Potentials are compared at 1e-4 of their scale: the logits are exact
float32 here, there is no stored bf16 kernel."""
import numpy as np
import pytest
import torch

from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import synth
from lot_testutil import check_slice, gpu_forward, oracle_slices

pytestmark = pytest.mark.gpu
SLICE = 3

CASES = [
    # B, H, n, r, iters, eps, key mask, clustered
    (1, 1, 1, 1, 3, 0.1, False, False),
    (1, 1, 16, 16, 2, 0.1, False, False),
    (2, 3, 197, 16, 10, 0.1, False, False),        # config 2
    (2, 12, 512, 32, 20, 0.05, True, False),       # config 3
    (1, 2, 256, 64, 10, 0.1, False, False),        # the widest pivot tile
    (1, 3, 250, 40, 5, 0.1, True, False),
    (1, 2, 512, 16, 7, 0.1, False, False),
    (1, 2, 300, 17, 4, 0.2, True, False),          # two tiles per warp, ragged
    (1, 2, 100, 33, 0, 0.1, False, False),         # no iteration
    (1, 1, 255, 64, 50, 0.1, False, False),
    (1, 2, 512, 32, 6, 0.01, False, True),         # peaked similarities
    (1, 2, 256, 64, 20, 0.01, True, True),
    (1, 4, 400, 8, 5, 0.02, False, True),
    (40, 8, 130, 24, 3, 0.1, True, False),         # 320 slices: more than one wave
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "B%d-H%d-n%d-r%d-T%d-eps%g-%s-%s" % (
    c[:6] + ("mask" if c[6] else "full", "peaked" if c[7] else "normal")))
def test_slice_path_matches_oracle(case):
    B, H, n, r, iters, eps, masked, peaked = case
    assert lot.lot_path(lot.LOT_BF16, B, H, n, 64, r, iters) == SLICE
    assert lot.lot_launch_count(lot.LOT_BF16, B, H, n, 64, r, iters) == 1
    x = synth.make(B, H, n, 64, r, seed=3000 + 7 * n + H, dtype=torch.bfloat16, eps=eps, iters=iters,
                   key_len_range=(max(1, n // 2), n) if masked else None, qk="mixture" if peaked else "normal")
    res = gpu_forward(x, want_g=True)
    assert res["status"] == 0
    assert np.isfinite(res["out"]).all()
    slices = sorted({(0, 0), (B // 2, H // 2), (B - 1, H - 1)})
    outs, g1s, g2s = oracle_slices(x, slices, return_potentials=True)
    worst = 0.0
    for (b, h), o, g1, g2 in zip(slices, outs, g1s, g2s):
        he, ee = check_slice(res["out"][b, h], o, 2e-2, f"slice {(b, h)}")
        worst = max(worst, ee)
        scale = max(1.0, np.abs(g1).max(), np.abs(g2).max())
        assert np.abs(res["g1"][b, h] - g1).max() <= 1e-4 * scale
        assert np.abs(res["g2"][b, h] - g2).max() <= 1e-4 * scale
    print(f"slice path {case}: worst elementwise {worst:.2e}")


def test_slice_path_key_lengths_one_and_zero():
    """One valid key: every query attends to it alone.  No valid key: zero output, flagged LOT_DEV_EMPTY."""
    x = synth.make(2, 2, 200, 64, 16, seed=3900, dtype=torch.bfloat16, eps=0.1, iters=5, key_len_range=(1, 1))
    x.key_len[1] = 0
    res = gpu_forward(x)
    assert res["status"] == lot.LOT_DEV_EMPTY
    v = x.v.float().double().numpy()
    for h in range(2):
        assert np.abs(res["out"][0, h] - v[0, h, 0][None, :]).max() <= 2e-2 * np.abs(v[0, h, 0]).max()
        assert not res["out"][1, h].any()


def test_slice_path_is_repeatable():
    x = synth.config(3, B=4)
    a = gpu_forward(x, want_g=True)
    b = gpu_forward(x, want_g=True)
    assert np.array_equal(a["out"], b["out"]) and np.array_equal(a["g1"], b["g1"]) and np.array_equal(a["g2"], b["g2"])
