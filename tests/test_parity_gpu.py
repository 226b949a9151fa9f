"""Parity of the CUDA path (through the C ABI) against the float64 CPU oracle on the same seeded,
dtype-rounded inputs.  Tolerances: max |out - ref| / max |ref| per (batch, head) slice <= 1e-4 for
float32 tensors and <= 2e-2 for bf16 tensors."""
import numpy as np
import pytest
import torch

from oracle import lot_oracle as O
from paper_2509_23436_b200 import binding as lot
from paper_2509_23436_b200 import synth

from lot_testutil import (TOL, check_slice, gpu_forward, head_err, oracle_all, oracle_slice, oracle_slices, to_dev,
                          worst_head_err)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


# ----------------------------------------------------------------------------- stage: cost
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape", [(1, 1, 64, 16, 8), (2, 3, 197, 64, 16), (1, 2, 300, 128, 100), (1, 1, 1, 8, 1),
                                   (1, 2, 130, 256, 256)])
def test_cost_matches_oracle(shape, dtype):
    B, H, n, d, r = shape
    x = synth.make(B, H, n, d, r, seed=11, dtype=dtype)
    C = lot.lot_cost(x.q.to(DEV), x.z.to(DEV)).cpu().double().numpy()
    f = x.f64()
    for b in range(B):
        for h in range(H):
            ref = O.cost(f["q"][b, h], f["z"][h])
            assert np.abs(C[b, h] - ref).max() <= 2e-6 * max(1.0, np.abs(ref).max())


# ----------------------------------------------------------------------------- stage: sinkhorn
@pytest.mark.parametrize("shape,eps,iters", [
    ((1, 1, 64, 8), 0.1, 50), ((2, 3, 197, 16), 0.1, 10), ((2, 2, 512, 32), 0.05, 20),
    ((1, 2, 1000, 64), 0.1, 10), ((1, 1, 777, 100), 0.1, 3), ((1, 1, 600, 256), 0.1, 5),
    ((1, 1, 50, 1), 0.1, 4), ((1, 1, 1, 8), 0.1, 2), ((1, 2, 300, 64), 0.1, 0),
])
def test_sinkhorn_matches_oracle(shape, eps, iters):
    B, H, n, r = shape
    g = torch.Generator().manual_seed(5)
    cost = torch.randn(B, H, n, r, generator=g)
    beta = torch.softmax(torch.randn(H, r, generator=g), -1)
    length = torch.randint(max(1, n // 2), n + 1, (B,), generator=g).to(torch.int32)
    for use_len in (False, True):
        ln = length.to(DEV) if use_len else None
        gg, ff, pp, ws = lot.lot_sinkhorn(cost.to(DEV), beta.to(DEV), ln, eps, iters, want_f=True, want_plan=True)
        torch.cuda.synchronize()
        assert lot.lot_device_status(ws) == 0
        for b in range(B):
            L = int(length[b]) if use_len else n
            m = np.zeros(n); m[:L] = 1.0 / L
            for h in range(H):
                g_ref, f_ref, P_ref = O.sinkhorn(cost[b, h].double().numpy(), beta[h].double().numpy(), m, eps, iters)
                P = pp[b, h].cpu().double().numpy()
                assert np.abs(P - P_ref).max() <= 1e-4 * P_ref.max()
                np.testing.assert_allclose(gg[b, h].cpu().double().numpy(), g_ref, atol=2e-5 * max(1, np.abs(g_ref).max()))
                fv = ff[b, h].cpu().double().numpy()
                np.testing.assert_allclose(fv[:L], f_ref[:L], atol=2e-5 * max(1, np.abs(f_ref[:L]).max()))
                assert np.all(np.isneginf(fv[L:])) and np.all(P[L:] == 0)


def test_sinkhorn_peaked_costs_small_eps_stays_finite():
    """Logits of several hundred: plain exp would overflow float32; column masses of far pivots
    underflow unless carried as (exponent, mantissa-sum) pairs."""
    x = synth.make(1, 2, 2048, 128, 64, seed=5003, eps=0.01, iters=20, qk="mixture")
    t = to_dev(x)
    cost = lot.lot_cost(t["q"], t["z"])
    assert float(cost.abs().max()) / 0.01 > 200
    gg, ff, pp, ws = lot.lot_sinkhorn(cost, t["beta"], None, 0.01, 20, want_f=True, want_plan=True)
    torch.cuda.synchronize()
    assert lot.lot_device_status(ws) == 0
    assert torch.isfinite(gg).all() and torch.isfinite(pp).all()
    for h in range(2):
        g_ref, _, P_ref = O.sinkhorn(cost[0, h].cpu().double().numpy(), x.beta[h].double().numpy(),
                                     np.full(2048, 1 / 2048), 0.01, 20)
        P = pp[0, h].cpu().double().numpy()
        assert np.abs(P - P_ref).max() <= 2e-3 * P_ref.max()
        assert np.abs(P.sum(0) - P_ref.sum(0)).max() <= 1e-3 * P_ref.sum(0).max()


# ----------------------------------------------------------------------------- whole forward, configs 1-3
def _check_full(x, want_g=True):
    res = gpu_forward(x, want_g=want_g)
    assert res["status"] == 0
    d = x.f64()
    ref, g1, g2, _ = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters,
                                     key_len=d["key_len"], return_potentials=True)
    err, worst_elem = 0.0, 0.0
    for b in range(ref.shape[0]):
        for h in range(ref.shape[1]):
            he, ee = check_slice(res["out"][b, h], ref[b, h], TOL[x.q.dtype], f"{x.name} {x.q.dtype} slice {(b, h)}")
            err, worst_elem = max(err, he), max(worst_elem, ee)
    print(f"{x.name} {x.q.dtype}: normwise {err:.3e}, elementwise {worst_elem:.3e}")
    if want_g:
        # potentials: float32 tensors 1e-4; bf16 tensors 1e-3, because passes 2..T of the fused bf16 path read the
        # Gibbs kernel exp(C/eps - rowmax) back as bf16 (relative rounding 2^-9 per entry, averaged over the tokens)
        gtol = 1e-4 if x.q.dtype == torch.float32 else 1e-3
        sc = max(1.0, np.abs(g1).max(), np.abs(g2).max())
        assert np.abs(res["g1"] - g1).max() <= gtol * sc and np.abs(res["g2"] - g2).max() <= gtol * sc
    return err


def test_config1_tiny_fp32():
    _check_full(synth.config(1))


def test_config1_named_entry_point_fp32():
    x = synth.config(1)
    t = to_dev(x)
    out = lot.lot_attention_fwd(t["q"], t["k"], t["v"], t["z"], t["beta"], x.eps, x.iters)
    torch.cuda.synchronize()
    assert lot.lot_device_status(None) == 0
    assert worst_head_err(out.cpu().double().numpy(), oracle_all(x)) <= 1e-4


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_config2_deit_tiny(dtype):
    _check_full(synth.config(2, dtype=dtype))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_config3_bert_base_with_key_mask(dtype):
    x = synth.config(3, dtype=dtype)
    assert x.key_len is not None and int(x.key_len.min()) >= 256
    _check_full(x)


# ----------------------------------------------------------------------------- config 4 (headline family)
@pytest.mark.parametrize("n", [4096, 16384])
def test_config4_long_context_bf16_all_heads(n):
    _check_full(synth.config(4, n=n), want_g=False)


def test_config4_n65536_all_heads_and_potentials():
    """The one length of config 4 whose stored Gibbs kernel (268 MB) does not stay in the L2."""
    x = synth.config(4, n=65536)
    res = gpu_forward(x, want_g=True)
    assert res["status"] == 0
    H = x.shape[1]
    outs, g1s, g2s = oracle_slices(x, [(0, h) for h in range(H)], return_potentials=True)
    for h in range(H):
        check_slice(res["out"][0, h], outs[h], 2e-2, f"n=65536 head {h}")
        sc = max(1.0, np.abs(g1s[h]).max(), np.abs(g2s[h]).max())
        assert np.abs(res["g1"][0, h] - g1s[h]).max() <= 1e-3 * sc
        assert np.abs(res["g2"][0, h] - g2s[h]).max() <= 1e-3 * sc


def test_config4_fp32_n4096():
    _check_full(synth.config(4, n=4096, dtype=torch.float32), want_g=False)


# ----------------------------------------------------------------------------- config 5 (rank / iteration stress): the whole grid
CFG5_SLICES = ((0, 0), (1, 3), (2, 5), (3, 7))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32], ids=["bf16", "f32"])
@pytest.mark.parametrize("eps", [0.1, 0.01])
@pytest.mark.parametrize("iters", [5, 20, 50])
@pytest.mark.parametrize("r", [16, 64, 128, 256])
def test_config5_stress_grid(r, iters, eps, dtype):
    """Every cell of config 5 (4 ranks x 3 iteration counts x 2 eps x 2 dtypes) at full size; the oracle checks four
    (batch, head) slices of each, the first and the last among them, and every output entry must be finite."""
    x = synth.config(5, r=r, iters=iters, eps=eps, dtype=dtype)
    res = gpu_forward(x)
    assert res["status"] == 0
    assert np.isfinite(res["out"]).all()
    refs = oracle_slices(x, CFG5_SLICES)
    for (b, h), ref in zip(CFG5_SLICES, refs):
        check_slice(res["out"][b, h], ref, TOL[dtype], f"r={r} T={iters} eps={eps} {dtype} slice {(b, h)}")


# ----------------------------------------------------------------------------- edge and degenerate cases
@pytest.mark.parametrize("shape", [(1, 1, 1, 8, 1), (1, 1, 1, 16, 8), (2, 2, 3, 8, 4), (1, 1, 65, 24, 7),
                                   (1, 3, 129, 40, 33), (1, 1, 257, 256, 256), (3, 1, 64, 16, 8)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ragged_and_degenerate_shapes(shape, dtype):
    B, H, n, d, r = shape
    x = synth.make(B, H, n, d, r, seed=77, dtype=dtype, eps=0.2, iters=4)
    _check_full(x)


def test_r1_gives_key_mean_and_iters0():
    x = synth.make(1, 2, 100, 16, 1, seed=3, eps=0.1, iters=3)
    res = gpu_forward(x)
    mean_v = x.v.double().numpy().mean(2, keepdims=True)
    assert np.abs(res["out"] - mean_v).max() < 1e-6
    x0 = synth.make(1, 2, 100, 16, 8, seed=4, eps=0.1, iters=0)
    _check_full(x0)


def test_empty_inputs_are_noops():
    z = torch.zeros(1, 8, 16, device=DEV)
    q = torch.zeros(0, 1, 4, 16, device=DEV)
    out, _ = lot.lot_attention_fwd_ex(q, q, q, z, torch.full((1, 8), 0.125, device=DEV), None, 0.1, 2)
    assert out.shape == q.shape
    q = torch.zeros(1, 1, 0, 16, device=DEV)
    out, _ = lot.lot_attention_fwd_ex(q, q, q, z, torch.full((1, 8), 0.125, device=DEV), None, 0.1, 2)
    assert out.numel() == 0


def test_device_status_flags_nonpositive_beta_and_empty_keys():
    x = synth.make(2, 1, 64, 16, 8, seed=9, eps=0.1, iters=2)
    t = to_dev(x)
    bad = t["beta"].clone(); bad[0, 3] = 0.0
    _, ws = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], bad, None, x.eps, x.iters)
    assert lot.lot_device_status(ws) & lot.LOT_DEV_NONFINITE
    kl = torch.tensor([0, 40], dtype=torch.int32, device=DEV)
    out, ws = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], kl, x.eps, x.iters)
    assert lot.lot_device_status(ws) & lot.LOT_DEV_EMPTY
    assert float(out[0].abs().max()) == 0.0 and torch.isfinite(out).all()
    # the same workspace is clean again on the next good call
    _, ws2 = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], None, x.eps, x.iters, ws=ws)
    assert lot.lot_device_status(ws2) == 0


def test_deterministic_and_workspace_reuse():
    x = synth.config(2)
    t = to_dev(x)
    a, ws = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], None, x.eps, x.iters)
    b, _ = lot.lot_attention_fwd_ex(t["q"], t["k"], t["v"], t["z"], t["beta"], None, x.eps, x.iters, ws=ws)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_metamorphic_on_gpu():
    """Permuting keys with their values, or pivots with their masses, or shifting all pivots,
    leaves the output unchanged (up to rounding); permuting queries permutes rows."""
    x = synth.make(1, 2, 333, 32, 12, seed=21, eps=0.15, iters=6)
    base = gpu_forward(x)["out"]
    g = torch.Generator().manual_seed(1)
    pk, pq, pz = torch.randperm(333, generator=g), torch.randperm(333, generator=g), torch.randperm(12, generator=g)
    y = synth.make(1, 2, 333, 32, 12, seed=21, eps=0.15, iters=6)
    y.k, y.v = x.k[:, :, pk].contiguous(), x.v[:, :, pk].contiguous()
    assert np.abs(gpu_forward(y)["out"] - base).max() < 1e-5
    y = synth.make(1, 2, 333, 32, 12, seed=21, eps=0.15, iters=6)
    y.q = x.q[:, :, pq].contiguous()
    assert np.abs(gpu_forward(y)["out"] - base[:, :, pq.numpy()]).max() < 1e-5
    y = synth.make(1, 2, 333, 32, 12, seed=21, eps=0.15, iters=6)
    y.z, y.beta = x.z[:, pz].contiguous(), x.beta[:, pz].contiguous()
    assert np.abs(gpu_forward(y)["out"] - base).max() < 1e-5
