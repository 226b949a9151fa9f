"""The resident tensor-core path (bf16 tensors, d = 64, r <= 64: the Gibbs kernel stays in tensor memory and shared
memory across the Sinkhorn iterations) against the float64 oracle, over the launch geometries it has: split mode
(one contiguous tile range per thread block, column partials exchanged through global memory), whole mode (whole
sequences per block, one or two at a time, several waves), spilled key tiles (a block with more than 12 key tiles),
key masks that leave blocks without key tiles, every padded pivot width, zero and one iteration.  The library
takes this path by default only where it measured faster; here the test hook selects it everywhere it can run.
Also: a problem the stored kernel cannot represent is recomputed by the streamed kernels, and a wait that cannot
end runs out, is reported, and leaves the workspace usable."""
import numpy as np
import pytest
import torch

from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import synth
from lot_testutil import check_slice, oracle_slices, to_dev

pytestmark = pytest.mark.gpu
RESIDENT = 2


@pytest.fixture
def resident_path():
    lot.lot_debug_hook(4, RESIDENT)
    yield
    lot.lot_debug_hook(4, -1)
    lot.lot_debug_hook(2, 0)
    lot.lot_debug_hook(1, -1)


def _forward(x, ws=None):
    t = to_dev(x)
    B, H, n, d, r = x.shape
    g1 = torch.empty(B, H, r, device="cuda:0")
    g2 = torch.empty(B, H, r, device="cuda:0")
    out, ws = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], t["key_len"], x.eps, x.iters,
                                       g1_out=g1, g2_out=g2, ws=ws)
    torch.cuda.synchronize()
    return dict(out=out.float().cpu().double().numpy(), g1=g1.cpu().double().numpy(), g2=g2.cpu().double().numpy(),
                status=lot.lot_device_status(ws), ws=ws)


def _check(x, res, slices):
    outs, g1s, g2s = oracle_slices(x, slices, return_potentials=True)
    for (b, h), o, g1, g2 in zip(slices, outs, g1s, g2s):
        check_slice(res["out"][b, h], o, 2e-2, f"{x.name} slice {(b, h)}")
        scale = max(1.0, np.abs(g1).max(), np.abs(g2).max())
        # the stored kernel is rounded to bf16 once: potentials to 1e-3 (see test_parity_gpu)
        assert np.abs(res["g1"][b, h] - g1).max() <= 1e-3 * scale
        assert np.abs(res["g2"][b, h] - g2).max() <= 1e-3 * scale


CASES = [
    # B, H, n, r, iters, eps, key mask
    (1, 1, 100, 64, 3, 0.1, False),        # one block, one tile
    (1, 1, 128, 64, 0, 0.1, False),        # no iteration: first pass, then the apply phases
    (1, 1, 300, 64, 1, 0.1, False),        # split over three blocks, one pivot update
    (2, 2, 300, 64, 5, 0.1, True),         # blocks whose key range lies beyond the mask
    (1, 3, 700, 32, 4, 0.1, False),
    (2, 3, 197, 16, 10, 0.1, False),
    (1, 3, 1700, 64, 4, 0.1, True),        # 14 tiles per sequence: spilled key tiles in whole mode
    (1, 200, 130, 48, 3, 0.2, True),       # more sequences than blocks: two per wave
    (1, 600, 130, 64, 2, 0.1, False),      # several waves
    (1, 2, 5000, 64, 4, 0.1, False),
    (1, 1, 20000, 64, 3, 0.1, False),      # every block shares the one slice
    (2, 8, 3000, 33, 6, 0.1, True),
    (1, 16, 4096, 64, 10, 0.1, False),
    (1, 16, 16384, 64, 10, 0.1, False),    # 14 + 14 tiles per block: the capacity of the path
    (16, 12, 512, 32, 20, 0.05, True),
    (32, 3, 197, 16, 10, 0.1, False),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "B%d-H%d-n%d-r%d-T%d-eps%g-%s" % (c[:6] + ("mask" if c[6] else "full",)))
def test_resident_path_matches_oracle(case, resident_path):
    B, H, n, r, iters, eps, masked = case
    assert lot.lot_path(lot.LOT_BF16, B, H, n, 64, r, iters) == RESIDENT
    x = synth.make(B, H, n, 64, r, seed=1000 + 7 * n + H, dtype=torch.bfloat16, eps=eps, iters=iters,
                   key_len_range=(max(1, n // 2), n) if masked else None)
    res = _forward(x)
    assert res["status"] == 0            # in particular: not recomputed by the streamed kernels
    assert np.isfinite(res["out"]).all()
    _check(x, res, sorted({(0, 0), (B // 2, H // 2), (B - 1, H - 1)}))


def test_resident_path_hands_unrepresentable_problems_to_the_streamed_kernels(resident_path):
    """Clustered tokens at eps = 0.01 spread the potentials over hundreds of binades: the call is flagged as
    recomputed and its results are the streamed kernels', within the same tolerances."""
    x = synth.make(1, 2, 2048, 64, 64, seed=15337, dtype=torch.bfloat16, eps=0.01, iters=6, qk="mixture")
    res = _forward(x)
    assert res["status"] == lot.LOT_DEV_RECOMPUTED
    _check(x, res, [(0, 0), (0, 1)])


def test_bitwise_repeatable(resident_path):
    x = synth.make(1, 4, 3000, 64, 64, seed=5, dtype=torch.bfloat16, eps=0.1, iters=5)
    a = _forward(x)
    b = _forward(x, ws=a["ws"])
    assert a["status"] == 0 and b["status"] == 0
    assert np.array_equal(a["out"], b["out"]) and np.array_equal(a["g1"], b["g1"])


def test_wait_that_cannot_end_times_out_and_the_workspace_stays_usable(resident_path):
    """Block 0 never publishes its first column partial (test hook), so the blocks that share its slice poll in vain:
    with the wait limit at 20 ms every block gives up, the call ends with LOT_DEV_TIMEOUT, nothing hangs, and the
    next call on the same workspace is clean and correct."""
    x = synth.make(1, 2, 3000, 64, 64, seed=8, dtype=torch.bfloat16, eps=0.1, iters=4)
    lot.lot_debug_hook(2, 20_000_000)
    lot.lot_debug_hook(1, 0)
    bad = _forward(x)
    assert bad["status"] & lot.LOT_DEV_TIMEOUT
    good = _forward(x, ws=bad["ws"])
    assert good["status"] == 0
    _check(x, good, [(0, 0), (0, 1)])
