"""The bounds-check build (liblot_debug.so: the same sources compiled with -DLOT_DEBUG, every checked global access of
the general-path and backward kernels states its buffer's extent, an access outside it is skipped and flagged
LOT_DEV_BOUNDS, never a trap) run once over tiny and odd-shaped cases, in a process of its own: no flag, results equal
to the regular build's bit for bit."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, torch
sys.path.insert(0, %r)
from paper_2509_23436_b200 import binding as lot, synth
assert (lot.lib().lot_version() >= 100000) == %s
dev = torch.device("cuda:0")
lot.lot_debug_hook(4, 0)                                # the general path everywhere
res = []
cases = [synth.config(1), synth.make(2, 2, 130, 40, 50, seed=11, dtype=torch.float32, eps=0.1, iters=4, key_len_range=(60, 130)),
         synth.make(1, 3, 197, 64, 16, seed=12, dtype=torch.bfloat16, eps=0.1, iters=5),
         synth.make(1, 1, 257, 128, 200, seed=13, dtype=torch.bfloat16, eps=0.05, iters=3)]
for x in cases:
    kl = None if x.key_len is None else x.key_len.to(dev)
    t = [v.to(dev) for v in (x.q, x.k, x.v, x.z, x.beta)]
    out, ws = lot.lot_attention_fwd_ex(*t, kl, x.eps, x.iters)
    torch.cuda.synchronize()
    assert lot.lot_device_status(ws) == 0, "forward flagged"
    g = lot.lot_attention_bwd(*t, kl, synth.cotangent(x).to(dev), x.eps, x.iters)
    torch.cuda.synchronize()
    assert lot.lot_device_status(g[5]) == 0, "backward flagged"
    res.append([out.cpu()] + [v.cpu() for v in g[:5]])
torch.save(res, sys.argv[1])
"""


def _run(lib, debug, path):
    env = dict(os.environ)
    if lib:
        env["LOT_LIBRARY"] = lib
    else:
        env.pop("LOT_LIBRARY", None)
    subprocess.run([sys.executable, "-c", CHILD % (ROOT, debug), path], check=True, env=env, cwd=ROOT, timeout=600)


def test_bounds_check_build_runs_clean_and_agrees(tmp_path):
    import torch
    dbg = os.path.join(ROOT, "paper_2509_23436_b200", "liblot_debug.so")
    if not os.path.exists(dbg):
        from paper_2509_23436_b200 import build
        build.build_lib(debug=True)
    a, b = str(tmp_path / "debug.pt"), str(tmp_path / "regular.pt")
    _run(dbg, True, a)
    _run(None, False, b)
    ra, rb = torch.load(a), torch.load(b)
    for ca, cb in zip(ra, rb):
        for ta, tb in zip(ca, cb):
            assert torch.equal(ta, tb)
