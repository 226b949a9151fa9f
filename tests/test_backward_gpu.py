"""Parity of lot_attention_bwd (Section "Learning": gradients through the two Sinkhorn problems, Eq. (1)-(2), and the
glued composition, Eq. (3)-(4)) with the float64 reverse sweep of the oracle, slice by slice, through the C ABI.

The oracle gradient is pinned on the CPU by central finite differences of the C oracle (test_oracle_pins.py).  A key
mask is the truncated problem for the oracle (a pinned equivalence); the rows of dk and dv beyond the key length must
come back as exact zeros.  Tolerances are those of the forward (1e-4 for float32 tensors, 2e-2 for bf16 tensors),
normwise and elementwise per slice: the backward runs in the same arithmetic as the forward general path (float64 for
float32 tensors, float32 for bf16 tensors with bf16-rounded dq, dk, dv)."""
import numpy as np
import pytest
import torch

from oracle import lot_oracle_grad as OG
from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import synth
from lot_testutil import TOL, check_slice

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16

# B, H, n, d, r, iters, eps, dtype, key mask
CASES = [
    (2, 2, 200, 64, 16, 5, 0.1, F32, False),
    (2, 3, 197, 64, 16, 10, 0.1, BF16, False),         # config 2's shape
    (2, 2, 300, 64, 32, 8, 0.05, F32, True),           # config 3's eps and mask
    (1, 2, 512, 64, 64, 3, 0.1, BF16, True),
    (1, 1, 130, 40, 50, 4, 0.1, F32, False),           # r not a multiple of 4, odd d
    (1, 2, 260, 128, 128, 2, 0.1, BF16, False),        # config 5's d; eight lanes per row
    (1, 1, 150, 32, 200, 2, 0.1, F32, False),          # sixteen lanes per row
    (1, 2, 129, 64, 8, 0, 0.1, F32, False),            # no iteration: plain softmax plans
    (1, 2, 129, 64, 8, 1, 0.1, BF16, False),
    (3, 2, 700, 64, 64, 12, 0.1, F32, True),           # several row chunks per problem
    (1, 1, 2048, 64, 64, 10, 0.1, BF16, False),
]


def oracle_grads(x, dout):
    """Oracle gradients: per-slice dq, dk, dv and the batch sums dz, dbeta."""
    d = x.f64()
    B, H, n, dd, r = x.shape
    do = dout.to(torch.float64).numpy()
    dq, dk, dv = (np.zeros((B, H, n, dd)) for _ in range(3))
    dz, dbeta = np.zeros((H, r, dd)), np.zeros((H, r))
    for b in range(B):
        kv = n if d["key_len"] is None else int(d["key_len"][b])
        a = np.full(n, 1.0 / n)
        bb = np.full(kv, 1.0 / kv)
        for h in range(H):
            fw = OG.head_forward(d["q"][b, h], d["k"][b, h, :kv], d["v"][b, h, :kv], d["z"][h], d["beta"][h], a, bb,
                                 x.eps, x.iters)
            g = OG.head_backward(fw, do[b, h])
            dq[b, h] = g["dq"]
            dk[b, h, :kv] = g["dk"]
            dv[b, h, :kv] = g["dv"]
            dz[h] += g["dz"]
            dbeta[h] += g["dbeta"]
    return dq, dk, dv, dz, dbeta


# config 5's peaked similarities (Gaussian-mixture queries and keys, d = 128), small eps
PEAKED = [
    (1, 2, 1024, 128, 64, 5, 0.05, BF16),
    (1, 1, 512, 128, 16, 20, 0.01, F32),
    (2, 1, 640, 128, 256, 5, 0.1, F32),
]


@pytest.mark.parametrize("B,H,n,d,r,iters,eps,dtype", PEAKED)
def test_backward_peaked_costs(B, H, n, d, r, iters, eps, dtype):
    run_case(synth.make(B, H, n, d, r, seed=7500 + n + r, dtype=dtype, eps=eps, iters=iters, qk="mixture"), False)


@pytest.mark.parametrize("B,H,n,d,r,iters,eps,dtype,masked", CASES)
def test_backward_matches_oracle(B, H, n, d, r, iters, eps, dtype, masked):
    run_case(synth.make(B, H, n, d, r, seed=7100 + n + r, dtype=dtype, eps=eps, iters=iters,
                        key_len_range=(n // 2, n) if masked else None), masked)


def run_case(x, masked):
    B, H, n, d, r = x.shape
    eps, iters, dtype = x.eps, x.iters, x.q.dtype
    dout = synth.cotangent(x)
    dev = torch.device("cuda:0")
    kl = None if x.key_len is None else x.key_len.to(dev)
    dq, dk, dv, dz, dbeta, ws = lot.lot_attention_bwd(x.q.to(dev), x.k.to(dev), x.v.to(dev), x.z.to(dev), x.beta.to(dev),
                                                      kl, dout.to(dev), eps, iters)
    torch.cuda.synchronize()
    assert lot.lot_device_status(ws) == 0
    rq, rk, rv, rz, rb = oracle_grads(x, dout)
    tol = TOL[dtype]
    got = {n_: t.float().cpu().double().numpy() for n_, t in (("dq", dq), ("dk", dk), ("dv", dv))}
    worst = {}
    for name, ref in (("dq", rq), ("dk", rk), ("dv", rv)):
        for b in range(B):
            for h in range(H):
                he, ee = check_slice(got[name][b, h], ref[b, h], tol, f"{name}[{b},{h}]")
                worst[name] = max(worst.get(name, 0.0), ee)
    if masked:
        for b in range(B):
            kv = int(x.key_len[b])
            assert not got["dk"][b, :, kv:].any() and not got["dv"][b, :, kv:].any(), "masked keys must get zero gradient"
    gz, gb = dz.cpu().double().numpy(), dbeta.cpu().double().numpy()
    for h in range(H):
        check_slice(gz[h], rz[h], tol, f"dz[{h}]")
        check_slice(gb[h][None, :], rb[h][None, :], tol, f"dbeta[{h}]")
    print(f"backward {x.meta} T={iters}: worst elementwise dq {worst['dq']:.2e} dk {worst['dk']:.2e} dv {worst['dv']:.2e}")


def test_backward_is_repeatable_and_checks_arguments():
    x = synth.make(1, 2, 300, 64, 32, seed=7300, dtype=BF16, eps=0.1, iters=4)
    dout = synth.cotangent(x)
    dev = torch.device("cuda:0")
    args = (x.q.to(dev), x.k.to(dev), x.v.to(dev), x.z.to(dev), x.beta.to(dev), None, dout.to(dev), 0.1, 4)
    first = lot.lot_attention_bwd(*args)
    second = lot.lot_attention_bwd(*args, ws=first[5])
    torch.cuda.synchronize()
    for a, b in zip(first[:5], second[:5]):
        assert torch.equal(a, b), "fixed summation order: two calls must agree bit for bit"
    with pytest.raises(lot.LotError):
        lot.lot_attention_bwd(*args[:7], -1.0, 4)
    with pytest.raises(lot.LotError):
        lot.lot_attention_bwd(*args, ws=torch.empty(1024, device=dev, dtype=torch.uint8))
    assert lot.lot_bwd_workspace_bytes(1, 2, 300, 64, 32, lot.LOT_BF16, 4) > 0
    assert lot.lot_bwd_workspace_bytes(1, 2, 300, 64, 32, 7, 4) == 0
