"""Shared helpers of the parity tests: run the CUDA path through the C ABI, run the CPU oracle on
chosen (batch, head) slices, and the error measure the tolerances are stated in."""
import numpy as np
import torch

from oracle import lot_oracle as O
from paper_2509_23436_b200 import binding as lot

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}


def to_dev(x):
    dev = torch.device("cuda:0")
    kl = None if x.key_len is None else x.key_len.to(dev)
    return dict(q=x.q.to(dev), k=x.k.to(dev), v=x.v.to(dev), z=x.z.to(dev), beta=x.beta.to(dev), key_len=kl)


def gpu_forward(x, want_g=False):
    t = to_dev(x)
    B, H, n, d, r = x.shape
    g1 = torch.empty(B, H, r, device="cuda:0") if want_g else None
    g2 = torch.empty(B, H, r, device="cuda:0") if want_g else None
    out, ws = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], t["key_len"], x.eps, x.iters,
                                       g1_out=g1, g2_out=g2)
    torch.cuda.synchronize()
    # LOT_DEV_RECOMPUTED is information, not an error: whichever tensor-core kernel produced the result, it is checked
    status = lot.lot_device_status(ws) & ~lot.LOT_DEV_RECOMPUTED
    res = dict(out=out.float().cpu().double().numpy(), status=status)
    if want_g:
        res["g1"] = g1.cpu().double().numpy()
        res["g2"] = g2.cpu().double().numpy()
    return res


def oracle_slice(x, b, h, return_potentials=False):
    """Oracle output of one (batch, head) slice, from the rounded inputs."""
    d = x.f64()
    kl = None if d["key_len"] is None else d["key_len"][b:b + 1]
    res = O.attention_fwd(d["q"][b:b + 1, h:h + 1], d["k"][b:b + 1, h:h + 1], d["v"][b:b + 1, h:h + 1],
                          d["z"][h:h + 1], d["beta"][h:h + 1], x.eps, x.iters, key_len=kl,
                          return_potentials=return_potentials)
    if return_potentials:
        return res[0][0, 0], res[1][0, 0], res[2][0, 0]
    return res[0, 0]


def oracle_all(x):
    d = x.f64()
    return O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters, key_len=d["key_len"])


def head_err(got, ref):
    """max |got - ref| / max |ref| over one (batch, head) slice: the measure the tolerances
    (1e-4 for float32 tensors, 2e-2 for bf16 tensors) are gated on."""
    return float(np.abs(got - ref).max() / np.abs(ref).max())


def worst_head_err(got, ref):
    B, H = ref.shape[:2]
    return max(head_err(got[b, h], ref[b, h]) for b in range(B) for h in range(H))


def elem_err(got, ref):
    """Elementwise relative error of one slice, max over entries of |got - ref| / max(|ref|, rms(ref)): entries
    smaller than the slice's root mean square are measured against that floor (an absolute error of tol * rms),
    so that a near-zero reference entry does not decide the figure.  Gated at the same tolerance as head_err."""
    floor = float(np.sqrt((ref ** 2).mean()))
    return float((np.abs(got - ref) / np.maximum(np.abs(ref), floor)).max())


def check_slice(got, ref, tol, what=""):
    """Both error figures of one (batch, head) slice against the tolerance; returns them."""
    he, ee = head_err(got, ref), elem_err(got, ref)
    assert he <= tol, f"{what}: normwise error {he:.3e} > {tol}"
    assert ee <= tol, f"{what}: elementwise error {ee:.3e} > {tol} (normwise {he:.3e})"
    return he, ee


def oracle_slices(x, slices, return_potentials=False):
    """Oracle results of several (batch, head) slices in one call (the oracle threads over slices)."""
    d = x.f64()
    bs = [b for b, _ in slices]
    hs = [h for _, h in slices]
    # one problem per requested slice: batch index runs over the list, one head each
    outs, g1s, g2s = [], [], []
    import concurrent.futures as cf

    def one(bh):
        b, h = bh
        kl = None if d["key_len"] is None else d["key_len"][b:b + 1]
        return O.attention_fwd(d["q"][b:b + 1, h:h + 1], d["k"][b:b + 1, h:h + 1], d["v"][b:b + 1, h:h + 1],
                               d["z"][h:h + 1], d["beta"][h:h + 1], x.eps, x.iters, key_len=kl, threads=1,
                               return_potentials=True)
    with cf.ThreadPoolExecutor(max_workers=min(len(slices), 8)) as ex:
        res = list(ex.map(one, list(zip(bs, hs))))
    for o, g1, g2, _ in res:
        outs.append(o[0, 0]); g1s.append(g1[0, 0]); g2s.append(g2[0, 0])
    if return_potentials:
        return outs, g1s, g2s
    return outs
