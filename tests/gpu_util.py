"""Helpers shared by the GPU parity tests: device upload, the checker run per (batch, head),
and the error metric max|Y_gpu - Y_ref| / max|Y_ref| per (batch, head)."""
import numpy as np
import torch

from oracle import favor_sharp as fs
from paper_2302_00787_b200 import binding as fb
from paper_2302_00787_b200 import workloads as wl

TOL = {"f32": 1e-4, "bf16": 1e-2}      # attention outputs, max relative error per (batch, head)
FIT_TOL = 1e-5                          # parameter fits, relative


def dev(a, dtype="f32"):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def host(t):
    t = t.detach()
    if t.dtype != torch.float64:
        t = t.float()
    return t.cpu().numpy().astype(np.float64)


def rel_err(got, ref):
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


def elem_err(got, ref, floor):
    """Element-wise relative error |got - ref| / |ref| over the entries with |ref| > floor * max|ref| (it is undefined
    near the zeros of ref): (largest, median)."""
    sel = np.abs(ref) > floor * np.max(np.abs(ref))
    e = np.abs(got - ref)[sel] / np.abs(ref)[sel]
    return float(e.max()), float(np.median(e))


# Element-wise bounds for attention outputs on entries above a tenth of the largest: bf16 outputs carry 2^-8 of
# rounding each and the tensor-core path's bf16 / fp16 features a few times that on small entries.
ELEM_TOL = {"f32": (1e-3, 1e-4), "bf16": (5e-2, 5e-3)}      # (largest, median)


def upload(w):
    Q, K, V = wl.make_qkv(w)
    Om = wl.make_omega(w)
    return (Q, K, V, Om), (dev(Q, w.dtype), dev(K, w.dtype), dev(V, w.dtype), dev(Om))


def gpu_fit(ctx, dQ, dK, d, variant, pool=fb.POOL_PER_BH):
    st = ctx.fsharp_stats(dQ, dK, pool=pool)
    pr = ctx.fsharp_fit_params(st, d, variant)
    assert ctx.status() == 0
    return st, pr


def oracle_unit(Q, K, V, Om, blob, d, b, h, causal, rows=None):
    p = fb.unpack_params(blob, d)
    return fs.favor_sharp_attention(Q[b, h], K[b, h], V[b, h], Om, p, causal=causal, rows=rows)
