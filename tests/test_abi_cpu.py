"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import build as lot_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    lot_build.build_lib()
    return lot.lib()


def test_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "lot.h")).read()
    declared = set(re.findall(r"LOT_API[^;(]*?\b(lot_\w+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in lot.h but not exported"
    assert declared == set(lot.SIGNATURES), "binding and header disagree on the entry points"
    assert L.lot_version() >= 100
    assert L.lot_status_string(0) == b"LOT_OK"


def test_workspace_queries_are_host_only(L):
    a = L.lot_workspace_bytes(1, 16, 16384, 64, 64, lot.LOT_F32)
    b = L.lot_workspace_bytes(1, 16, 65536, 64, 64, lot.LOT_F32)
    assert 0 < a < b
    assert a % 256 == 0
    # the fused bf16 path stores one bf16 Gibbs kernel per side, not float64 similarities, logits and row sums
    assert 0 < L.lot_workspace_bytes(1, 16, 16384, 64, 64, lot.LOT_BF16) < a // 3
    # and nothing of size n x r for r <= 32
    assert 0 < L.lot_workspace_bytes(1, 16, 16384, 64, 32, lot.LOT_BF16) < a // 16
    assert L.lot_launch_count(lot.LOT_BF16, 1, 16, 16384, 64, 64, 10) > 0
    assert L.lot_launch_count(lot.LOT_F32, 1, 16, 16384, 64, 64, 10) == 15 and L.lot_path(lot.LOT_F32, 1, 16, 16384, 64, 64, 10) == 0
    assert L.lot_workspace_bytes(1, 16, 16384, 64, 300, lot.LOT_BF16) == 0      # r too large
    assert L.lot_workspace_bytes(1, 16, 16384, 60, 64, lot.LOT_BF16) == 0       # d % 8 != 0
    assert L.lot_sinkhorn_workspace_bytes(2, 3, 100, 16) > 0
    assert L.lot_sinkhorn_workspace_bytes(2, 3, 100, 0) == 0


def test_bad_arguments_return_status_without_a_device(L):
    p = ctypes.c_void_p(4096)          # aligned dummy, never dereferenced on these paths
    odd = ctypes.c_void_p(4100)
    assert L.lot_cost(None, p, 0, 1, 1, 8, 16, 8, p, None) == 1
    assert L.lot_cost(odd, p, 0, 1, 1, 8, 16, 8, p, None) == 1
    assert L.lot_cost(p, p, 7, 1, 1, 8, 16, 8, p, None) == 1
    assert L.lot_cost(p, p, 0, 1, 1, 8, 12, 8, p, None) == 2
    assert L.lot_cost(p, p, 0, 1, 1, 8, 16, 257, p, None) == 2
    assert L.lot_cost(p, p, 0, 0, 1, 8, 16, 8, p, None) == 0          # empty batch: no-op
    assert L.lot_cost(p, p, 0, 1, 1, 0, 16, 8, p, None) == 0          # empty sequence: no-op
    # sinkhorn: eps, iters, workspace
    assert L.lot_sinkhorn(p, p, None, 1, 1, 8, 8, 0.0, 1, p, None, None, p, 1 << 20, None) == 1
    assert L.lot_sinkhorn(p, p, None, 1, 1, 8, 8, float("nan"), 1, p, None, None, p, 1 << 20, None) == 1
    assert L.lot_sinkhorn(p, p, None, 1, 1, 8, 8, 0.1, -1, p, None, None, p, 1 << 20, None) == 1
    assert L.lot_sinkhorn(p, p, None, 1, 1, 8, 8, 0.1, 1, p, None, None, None, 0, None) == 3
    assert L.lot_sinkhorn(p, p, None, 1, 1, 8, 8, 0.1, 1, p, None, None, p, 16, None) == 3
    # attention
    args = [p, p, p, p, p, None, 0, 1, 1, 8, 16, 8]
    assert L.lot_attention_fwd_ex(*args, 0.1, 1, p, None, None, p, 16, None) == 3
    assert L.lot_attention_fwd_ex(*args, -1.0, 1, p, None, None, p, 1 << 24, None) == 1
    args[6] = 3
    assert L.lot_attention_fwd_ex(*args, 0.1, 1, p, None, None, p, 1 << 24, None) == 1
    assert L.lot_device_status(None, None, None) == 1


def test_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros(1, 1, 8, 16)
    z = torch.zeros(1, 8, 16)
    with pytest.raises(lot.LotError):
        lot.lot_cost(x, z)
