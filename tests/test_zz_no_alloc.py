"""lot_sinkhorn_static: the Sinkhorn solve for callers that cannot allocate device memory (an
allocator-owning framework, a latency-critical loop, a plug-in handed tensors but no allocator).
Its scratch is a fixed array inside the library, so it must give what lot_sinkhorn gives on a
caller-provided workspace, call after call, although every call reuses the same array and finds
the previous call's leftovers in it.  The file name sorts last so that pytest collects it last: a run that stops at
the first failure (-x) has then already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import lot_oracle as O
from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import build as lot_build

DEV = "cuda:0"


def _problem(seed, B, H, n, r, with_len):
    g = torch.Generator().manual_seed(seed)
    cost = torch.randn(B, H, n, r, generator=g)
    beta = torch.softmax(torch.randn(H, r, generator=g), -1)
    length = torch.randint(max(1, n // 2), n + 1, (B,), generator=g).to(torch.int32) if with_len else None
    return cost.to(DEV), beta.to(DEV), None if length is None else length.to(DEV)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_on_consecutive_calls():
    # two calls in a row on different problems: the second one starts from the first one's leftovers
    for seed, shape, eps, iters, with_len in ((1, (2, 3, 700, 32), 0.1, 8, False), (2, (1, 2, 333, 64), 0.05, 12, True)):
        B, H, n, r = shape
        cost, beta, length = _problem(seed, B, H, n, r, with_len)
        assert lot.lot_sinkhorn_workspace_bytes(B, H, n, r) <= lot.LOT_STATIC_SCRATCH_BYTES
        g_ref, f_ref, p_ref, ws = lot.lot_sinkhorn(cost, beta, length, eps, iters, want_f=True, want_plan=True)
        g = torch.empty(B, H, r, device=DEV)
        f = torch.empty(B, H, n, device=DEV)
        plan = torch.empty(B, H, n, r, device=DEV)
        status = torch.full((1,), -1, device=DEV, dtype=torch.int32)
        lot.lot_sinkhorn_static(cost, beta, length, eps, iters, g, f, plan, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and lot.lot_device_status(ws) == 0
        # same kernels, same fixed reduction order: the parity tests' tolerance is met with room to spare
        assert (plan - p_ref).abs().max() <= 1e-4 * p_ref.max()
        torch.testing.assert_close(g, g_ref, rtol=0, atol=2e-5 * max(1.0, float(g_ref.abs().max())))
        fin = torch.isfinite(f_ref)
        assert torch.equal(fin, torch.isfinite(f))
        torch.testing.assert_close(f[fin], f_ref[fin], rtol=0, atol=2e-5 * max(1.0, float(f_ref[fin].abs().max())))
    # the second problem once more against the CPU oracle, so that this file stands without lot_sinkhorn
    for b in range(B):
        L = int(length[b])
        m = np.zeros(n); m[:L] = 1.0 / L
        for h in range(H):
            g_o, _, P_o = O.sinkhorn(cost[b, h].cpu().double().numpy(), beta[h].cpu().double().numpy(), m, eps, iters)
            assert np.abs(plan[b, h].cpu().double().numpy() - P_o).max() <= 1e-4 * P_o.max()
            np.testing.assert_allclose(g[b, h].cpu().double().numpy(), g_o, atol=2e-5 * max(1, np.abs(g_o).max()))


@pytest.mark.gpu
def test_static_scratch_calls_allocate_nothing_and_follow_their_stream():
    """What the entry point is for: after the first call has looked the array up, further calls leave the amount of
    free device memory unchanged; and a call given a side stream runs on that stream."""
    B, H, n, r = 2, 2, 500, 32
    cost, beta, _ = _problem(3, B, H, n, r, False)
    g = torch.empty(B, H, r, device=DEV)
    plan = torch.empty(B, H, n, r, device=DEV)
    lot.lot_sinkhorn_static(cost, beta, None, 0.1, 5, g, None, plan)
    torch.cuda.synchronize()
    want = plan.clone()
    side = torch.cuda.Stream()

    def rounds(k):
        for _ in range(k):
            plan.zero_()
            side.wait_stream(torch.cuda.current_stream())
            lot.lot_sinkhorn_static(cost, beta, None, 0.1, 5, g, None, plan, stream=side)
            side.synchronize()
            assert torch.equal(plan, want)

    rounds(1)            # torch's own caching allocator and the side stream have settled after this
    free0 = torch.cuda.mem_get_info()[0]
    rounds(5)
    assert torch.cuda.mem_get_info()[0] == free0


def test_static_scratch_rejects_problems_beyond_its_size():
    lot_build.build_lib()
    L = lot.lib()
    p = ctypes.c_void_p(4096)      # aligned dummy; the size check comes before any device work
    assert L.lot_sinkhorn_workspace_bytes(4, 16, 65536, 64) > lot.LOT_STATIC_SCRATCH_BYTES
    assert L.lot_sinkhorn_static(p, p, None, 4, 16, 65536, 64, 0.1, 1, p, None, None, None, None) == 3
    assert b"WORKSPACE" in L.lot_status_string(3)


def test_static_scratch_checks_arguments_before_any_device_work():
    """The same refusals as lot_sinkhorn, in the same order, on a machine with no device at all."""
    lot_build.build_lib()
    L = lot.lib()
    p, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    assert L.lot_sinkhorn_static(p, p, None, 1, 1, 8, 8, 0.0, 1, p, None, None, None, None) == 1      # eps
    assert L.lot_sinkhorn_static(p, p, None, 0, 1, 8, 8, -1.0, 1, p, None, None, None, None) == 1     # eps, empty batch
    assert L.lot_sinkhorn_static(p, p, None, 1, 1, 8, 8, 0.1, -1, p, None, None, None, None) == 1     # iters
    assert L.lot_sinkhorn_static(None, p, None, 1, 1, 8, 8, 0.1, 1, p, None, None, None, None) == 1   # null cost
    assert L.lot_sinkhorn_static(p, p, None, 1, 1, 8, 8, 0.1, 1, odd, None, None, None, None) == 1    # misaligned g
    assert L.lot_sinkhorn_static(p, p, None, 1, 1, 8, 8, 0.1, 1, p, None, None, ctypes.c_void_p(4098), None) == 1
    assert L.lot_sinkhorn_static(p, p, None, 0, 1, 8, 8, 0.1, 1, p, None, None, None, None) == 0      # empty batch
