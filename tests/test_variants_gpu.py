"""lot_attention_fwd_var against the float64 oracle: cross-attention (nq != nk), arbitrary token weights (with zero
weights), warm start from exported potentials, and the [CLS] softmax row of Eq. (5), for float32 and bf16 tensors."""
import numpy as np
import pytest
import torch

from oracle import lot_oracle as O
from paper_2509_23436_b200 import binding as lot
from lot_testutil import TOL, check_slice

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw(B, H, nq, nk, d, r, seed, dtype):
    g = torch.Generator().manual_seed(seed)
    rn = lambda *s: torch.randn(*s, generator=g)
    q, k, v = (rn(B, H, nq, d) * d ** -0.5).to(dtype), (rn(B, H, nk, d) * d ** -0.5).to(dtype), (rn(B, H, nk, d) * d ** -0.5).to(dtype)
    z = rn(H, r, d)
    beta = torch.softmax(rn(H, r), -1)
    a = torch.rand(B, H, nq, generator=g) + 0.05
    b = torch.rand(B, H, nk, generator=g) + 0.05
    if nq > 2:
        a[:, :, nq // 3] = 0.0                  # a query and a key without weight
    b[:, :, nk // 2] = 0.0
    a = a / a.sum(-1, keepdim=True)
    b = b / b.sum(-1, keepdim=True)
    return q, k, v, z, beta, a, b


def _np(t):
    return t.to(torch.float64).numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("shape", [(2, 2, 150, 333, 32, 12), (1, 3, 700, 129, 64, 64), (1, 1, 1, 5, 8, 3)])
def test_cross_attention_with_token_weights(shape, dtype):
    B, H, nq, nk, d, r = shape
    q, k, v, z, beta, a, b = _draw(B, H, nq, nk, d, r, 31, dtype)
    eps, iters = 0.2, 7
    g1 = torch.empty(B, H, r, device=DEV); g2 = torch.empty(B, H, r, device=DEV)
    out, ws = lot.lot_attention_fwd_var(q.to(DEV), k.to(DEV), v.to(DEV), z.to(DEV), beta.to(DEV), eps, iters,
                                        a=a.to(DEV), b=b.to(DEV), g1_out=g1, g2_out=g2)
    torch.cuda.synchronize()
    assert lot.lot_device_status(ws) == 0
    got = out.float().cpu().double().numpy()
    for bb in range(B):
        for h in range(H):
            ref = O.head_x(_np(q[bb, h]), _np(k[bb, h]), _np(v[bb, h]), _np(z[h]), _np(beta[h]), _np(a[bb, h]), _np(b[bb, h]), eps, iters)
            if nq > 1:
                check_slice(got[bb, h], ref["out"], TOL[dtype], f"slice {(bb, h)}")
            else:
                assert np.abs(got[bb, h] - ref["out"]).max() <= TOL[dtype] * max(np.abs(ref["out"]).max(), 1e-3)
            gtol = 1e-4 if dtype == torch.float32 else 1e-3
            sc = max(1.0, np.abs(ref["g1"]).max(), np.abs(ref["g2"]).max())
            assert np.abs(g1[bb, h].cpu().double().numpy() - ref["g1"]).max() <= gtol * sc
            assert np.abs(g2[bb, h].cpu().double().numpy() - ref["g2"]).max() <= gtol * sc
            assert nq <= 2 or np.all(got[bb, h, nq // 3] == 0.0)       # the weightless query's row


def test_uniform_variant_equals_the_plain_entry_point():
    from paper_2509_23436_b200 import synth
    x = synth.make(2, 2, 300, 32, 12, seed=4, eps=0.15, iters=6, key_len_range=(150, 300))
    t = {k_: getattr(x, k_).to(DEV) for k_ in ("q", "k", "v", "z", "beta", "key_len")}
    a, _ = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], t["key_len"], x.eps, x.iters)
    b, _ = lot.lot_attention_fwd_var(t["q"], t["k"], t["v"], t["z"], t["beta"], x.eps, x.iters, key_len=t["key_len"])
    torch.cuda.synchronize()
    assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_warm_start_continues_the_iteration(dtype):
    B, H, nq, nk, d, r = 1, 2, 257, 257, 32, 16
    q, k, v, z, beta, _, _ = _draw(B, H, nq, nk, d, r, 9, dtype)
    dq, dk, dv, dz, db = (t.to(DEV) for t in (q, k, v, z, beta))
    g1 = torch.empty(B, H, r, device=DEV); g2 = torch.empty(B, H, r, device=DEV)
    lot.lot_attention_fwd_var(dq, dk, dv, dz, db, 0.2, 4, g1_out=g1, g2_out=g2)
    h1 = torch.empty_like(g1); h2 = torch.empty_like(g2)
    cont, _ = lot.lot_attention_fwd_var(dq, dk, dv, dz, db, 0.2, 5, g1_in=g1, g2_in=g2, g1_out=h1, g2_out=h2)
    full, _ = lot.lot_attention_fwd_var(dq, dk, dv, dz, db, 0.2, 9)
    torch.cuda.synchronize()
    u = np.full(nq, 1 / nq)
    for h in range(H):
        ref = O.head_x(_np(q[0, h]), _np(k[0, h]), _np(v[0, h]), _np(z[h]), _np(beta[h]), u, u, 0.2, 9)
        check_slice(cont[0, h].float().cpu().double().numpy(), ref["out"], TOL[dtype], f"continued, head {h}")
        check_slice(full[0, h].float().cpu().double().numpy(), ref["out"], TOL[dtype], f"from zero, head {h}")
        assert np.abs(h1[0, h].cpu().double().numpy() - ref["g1"]).max() <= 1e-3 * max(1.0, np.abs(ref["g1"]).max())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("masked", [False, True])
def test_cls_softmax_row(dtype, masked):
    B, H, n, d, r = 2, 3, 197, 64, 16
    q, k, v, z, beta, _, _ = _draw(B, H, n, n, d, r, 17, dtype)
    key_len = torch.tensor([150, 197], dtype=torch.int32) if masked else None
    tau = 1.5
    out, ws = lot.lot_attention_fwd_var(q.to(DEV), k.to(DEV), v.to(DEV), z.to(DEV), beta.to(DEV), 0.1, 10,
                                        key_len=None if key_len is None else key_len.to(DEV), cls=True, cls_tau=tau)
    torch.cuda.synchronize()
    assert lot.lot_device_status(ws) == 0
    got = out.float().cpu().double().numpy()
    for bb in range(B):
        for h in range(H):
            ref = O.head_cls(_np(q[bb, h]), _np(k[bb, h]), _np(v[bb, h]), _np(z[h]), _np(beta[h]), 0.1, 10, tau,
                             key_len=None if key_len is None else int(key_len[bb]))
            check_slice(got[bb, h], ref, TOL[dtype], f"cls slice {(bb, h)}")
            assert np.abs(got[bb, h, 0] - ref[0]).max() <= TOL[dtype] * np.abs(ref[0]).max()


def test_variant_arguments_are_checked():
    z = torch.zeros(1, 4, 8, device=DEV); beta = torch.full((1, 4), 0.25, device=DEV)
    q = torch.zeros(1, 1, 6, 8, device=DEV); k = torch.zeros(1, 1, 9, 8, device=DEV)
    a = torch.full((1, 1, 6), 1 / 6, device=DEV)
    with pytest.raises(lot.LotError):                       # the [CLS] treatment fixes the weights itself
        lot.lot_attention_fwd_var(q, k, k, z, beta, 0.1, 2, a=a, cls=True, cls_tau=1.0)
    with pytest.raises(lot.LotError):
        lot.lot_attention_fwd_var(q, k, k, z, beta, 0.1, 2, cls=True, cls_tau=0.0)
