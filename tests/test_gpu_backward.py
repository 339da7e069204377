"""GPU parity of the backward pass: dQ, dK, dV from fsharp_attend_backward (through the C ABI) against the fp64
checker's vector-Jacobian product on the same seeded inputs, Omega and fitted parameters.  Metric and tolerances as
for the attention outputs: max|g_gpu - g_ref| / max|g_ref| per (batch, head), 1e-4 (fp32) / 1e-2 (bf16)."""
import numpy as np
import pytest
import torch

from oracle import favor_sharp as fs
from paper_2302_00787_b200 import binding as fb
from paper_2302_00787_b200 import workloads as wl
from tests.gpu_util import TOL, dev, gpu_fit, host, rel_err, upload

pytestmark = pytest.mark.gpu

W = wl.WORKLOADS


@pytest.fixture(scope="module")
def ctx():
    c = fb.Context(0)
    yield c
    c.close()


def cotangent(w, seed, L=None):
    rng = np.random.default_rng(seed)
    dY = rng.standard_normal((w.B, w.H, L or w.L, w.dv))
    return wl.bf16_round(dY) if w.dtype == "bf16" else dY.astype(np.float32).astype(np.float64)


def ddev(dY, dtype="f32"):
    return dev(dY.astype(np.float32), dtype)


def cases():
    return [
        W["cfg1"],                                                                     # fp32, one tile
        W["cfg1"].scaled(L=17, variant="posrf", d=32, dv=16, M=48),                    # ragged everything
        W["cfg2"].scaled(B=2, H=2, L=300),                                             # bf16, ragged tail
        W["cfg3b"].scaled(B=1, H=2, L=200),                                            # dense C (ADERF)
        W["cfg3"].scaled(B=1, H=2, L=512),                                             # causal, four chunks
        W["cfg1"].scaled(L=192, causal=True, chunk=64, variant="gerf"),                # fp32 causal
        W["cfg1"].scaled(L=256, causal=True, chunk=128, variant="aderf", d=32, dv=16, M=64),
        W["cfg5"].scaled(B=1, H=1, L=512, outlier_frac=0.1),                           # d = dv = 128, M = 512, chunk 256
    ]


def check(w, Q, K, V, dY, Om, prh, grads, qk_scale=1.0, omega_of=None, group_of=None):
    gQ, gK, gV = (host(g) for g in grads)
    for b in range(w.B):
        for h in range(w.H):
            g = b * w.H + h if group_of is None else group_of(b, h)
            p = fb.unpack_params(prh[g], w.d)
            om = Om if omega_of is None else omega_of(h)
            rQ, rK, rV = fs.favor_sharp_attention_vjp(Q[b, h], K[b, h], V[b, h], dY[b, h], om, p, causal=w.causal,
                                                      qk_scale=qk_scale)
            for name, got, ref in (("dQ", gQ[b, h], rQ), ("dK", gK[b, h], rK), ("dV", gV[b, h], rV)):
                assert rel_err(got, ref) < TOL[w.dtype], (name, b, h, rel_err(got, ref))


@pytest.mark.parametrize("w", cases(), ids=lambda w: f"{w.name}-L{w.L}-{w.variant}-{'causal' if w.causal else 'bidir'}")
def test_backward_matches_checker(ctx, w):
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    dY = cotangent(w, 5)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    grads = ctx.fsharp_attend_backward(dQ, dK, dV, ddev(dY, w.dtype), dOm, pr, causal=w.causal, chunk=w.chunk)
    assert ctx.status() == 0
    check(w, Q, K, V, dY, Om, pr.cpu().numpy(), grads)


def test_backward_unequal_lengths_and_query_key_scale(ctx):
    w = W["cfg1"].scaled(L=200, d=32, dv=16, M=64, variant="aderf")
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    Lk = 77
    K, V, dK, dV = K[:, :, :Lk], V[:, :, :Lk], dK[:, :, :Lk].contiguous(), dV[:, :, :Lk].contiguous()
    dY = cotangent(w, 6)
    s = 0.8
    st = ctx.fsharp_stats(dQ, dK, qk_scale=s)
    pr = ctx.fsharp_fit_params(st, w.d, w.variant)
    grads = ctx.fsharp_attend_backward(dQ, dK, dV, ddev(dY), dOm, pr, qk_scale=s)
    assert ctx.status() == 0
    check(w, Q, K, V, dY, Om, pr.cpu().numpy(), grads, qk_scale=s)


def test_backward_strided_layout_per_head_omega_and_pooling(ctx):
    w = W["cfg2"].scaled(B=2, H=3, L=256)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    OmH = np.stack([wl.orthogonal_omega(w.M, w.d, 77 + h) for h in range(w.H)])
    dY = cotangent(w, 7)
    st = ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD)
    pr = ctx.fsharp_fit_params(st, w.d, "sderf")
    tr = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)     # [B, L, H, *] storage
    grads = ctx.fsharp_attend_backward(tr(dQ), tr(dK), tr(dV), tr(ddev(dY, "bf16")), dev(OmH), pr, pool=fb.POOL_PER_HEAD)
    assert ctx.status() == 0
    assert all(not g.is_contiguous() for g in grads)
    check(w, Q, K, V, dY, None, pr.cpu().numpy(), grads, omega_of=lambda h: OmH[h], group_of=lambda b, h: h)


def test_backward_chunk_size_is_immaterial_and_no_gradient_from_the_future(ctx):
    w = W["cfg3"].scaled(B=1, H=1, L=512)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    dY = cotangent(w, 8)
    dY[:, :, 300:] = 0.0                                     # cotangent on the first 300 rows only
    ref = [host(g) for g in ctx.fsharp_attend_backward(dQ, dK, dV, ddev(dY, "bf16"), dOm, pr, causal=True, chunk=128)]
    assert np.all(ref[0][:, :, 300:] == 0) and np.all(ref[1][:, :, 300:] == 0) and np.all(ref[2][:, :, 300:] == 0)
    for ch in (64, 256):
        got = [host(g) for g in ctx.fsharp_attend_backward(dQ, dK, dV, ddev(dY, "bf16"), dOm, pr, causal=True, chunk=ch)]
        for a, b in zip(got, ref):
            assert rel_err(a, b) < 1e-2
    assert ctx.status() == 0


def test_backward_argument_checks(ctx):
    w = W["cfg1"].scaled(L=100)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    dY = ddev(cotangent(w, 9))
    with pytest.raises(fb.FsharpError) as e:
        ctx.fsharp_attend_backward(dQ, dK, dV, dY, dOm, pr, causal=True, chunk=64)        # 64 does not divide 100
    assert e.value.code == -2
    with pytest.raises(fb.FsharpError) as e:
        ctx.fsharp_attend_backward(dQ, dK[:, :, :0], dV[:, :, :0], dY, dOm, pr)           # no key
    assert e.value.code == -2
    with pytest.raises(fb.FsharpError) as e:
        flat = torch.empty(dY.numel() + 1, device="cuda")[1:].view(dY.shape)
        ctx.fsharp_attend_backward(dQ, dK, dV, flat, dOm, pr)                            # misaligned cotangent
    assert e.value.code == -3
    assert ctx.status() == 0
