"""GPU parity: every stage of the CUDA path, called through the C ABI, against the fp64
checker on the same seeded inputs and the same Omega.  Tolerances: attention outputs 1e-4
(fp32) / 1e-2 (bf16) max relative error per (batch, head); fits 1e-5 relative on the
rotation-invariant quantities (the literal B of Theorems 4.2/4.3 is one of many solutions)."""
import numpy as np
import pytest
import torch

from oracle import favor_sharp as fs
from paper_2302_00787_b200 import binding as fb
from paper_2302_00787_b200 import workloads as wl
from tests.gpu_util import ELEM_TOL, FIT_TOL, TOL, dev, elem_err, gpu_fit, host, oracle_unit, rel_err, upload

pytestmark = pytest.mark.gpu

W = wl.WORKLOADS


@pytest.fixture(scope="module")
def ctx():
    c = fb.Context(0)
    yield c
    c.close()


def small_cases():
    return [
        W["cfg1"],
        W["cfg2"].scaled(B=2, H=2, L=300),                       # ragged tail: 300 = 2*128 + 44
        W["cfg3"].scaled(B=1, H=2, L=512),
        W["cfg3b"].scaled(B=1, H=2, L=200),
        W["cfg5"].scaled(B=1, H=2, L=1024, outlier_frac=0.1),
        W["cfg1"].scaled(L=64, causal=True, chunk=64, variant="gerf"),
        W["cfg1"].scaled(L=17, variant="posrf", d=32, dv=16, M=48),
    ]


# ------------------------------------------------------------------ stats
@pytest.mark.parametrize("w", small_cases()[:5], ids=lambda w: w.name)
def test_stats_match_definition(ctx, w):
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    st = host(ctx.fsharp_stats(dQ, dK))
    d = w.d
    for b in range(w.B):
        for h in range(w.H):
            ref = fs.set_statistics(Q[b, h], K[b, h])
            g = st[b * w.H + h]
            M1, M2 = g[: d * d].reshape(d, d), g[d * d: 2 * d * d].reshape(d, d)
            scale = np.abs(ref["M1"]).max()
            assert np.abs(M1 - ref["M1"]).max() < 2e-6 * scale
            assert np.abs(M2 - ref["M2"]).max() < 2e-6 * scale
            assert np.abs(g[2 * d * d: 2 * d * d + d] - ref["mu4"]).max() < 2e-6
            assert np.abs(g[2 * d * d + d: 2 * d * d + 2 * d] - ref["mu5"]).max() < 2e-6


def test_stats_pooled_over_batch_and_strided(ctx):
    w = W["cfg2"].scaled(B=3, H=2, L=160)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    st = host(ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD))
    assert st.shape[0] == w.H
    for h in range(w.H):
        ref = fs.set_statistics(Q[:, h].reshape(-1, w.d), K[:, h].reshape(-1, w.d))
        assert np.abs(st[h][: w.d * w.d].reshape(w.d, w.d) - ref["M1"]).max() < 2e-6 * np.abs(ref["M1"]).max()
    # [B, L, H, d] storage viewed as [B, H, L, d]
    dQs = dQ.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    dKs = dK.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not dQs.is_contiguous()
    st2 = host(ctx.fsharp_stats(dQs, dKs, pool=fb.POOL_PER_HEAD))
    assert np.abs(st2 - st).max() < 1e-12


@pytest.mark.parametrize("name", ["cfg2", "cfg5"])
def test_stats_tensor_core_path_matches_simt_and_definition(ctx, name):
    """bf16, d = 64 and d = 128 (four 64 x 64 blocks over the column halves) take the tensor-core Gram kernel: several
    tiles, a ragged tail, unequal query and key lengths, pooled and per-(batch, head) groups, and a query/key scale."""
    w = W[name].scaled(B=2, H=3, L=1000)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    dKs, Ks = dK[:, :, :333], K[:, :, :333]
    for pool in (fb.POOL_PER_BH, fb.POOL_PER_HEAD):
        st = host(ctx.fsharp_stats(dQ, dKs, pool=pool, qk_scale=0.75))
        ctx.set_impl(fb.IMPL_SIMT)
        try:
            st_simt = host(ctx.fsharp_stats(dQ, dKs, pool=pool, qk_scale=0.75))
        finally:
            ctx.set_impl(fb.IMPL_AUTO)
        assert ctx.status() == 0
        assert np.abs(st - st_simt).max() < 2e-6 * np.abs(st_simt).max()
        d = w.d
        for g in range(st.shape[0]):
            if pool == fb.POOL_PER_BH:
                b, h = divmod(g, w.H)
                ref = fs.set_statistics(0.75 * Q[b, h], 0.75 * Ks[b, h])
            else:
                ref = fs.set_statistics(0.75 * Q[:, g].reshape(-1, d), 0.75 * Ks[:, g].reshape(-1, d))
            for name, lo in (("M1", 0), ("M2", d * d)):
                assert np.abs(st[g][lo: lo + d * d].reshape(d, d) - ref[name]).max() < 2e-6 * np.abs(ref[name]).max()
            assert np.abs(st[g][2 * d * d: 2 * d * d + d] - ref["mu4"]).max() < 2e-6
            assert np.abs(st[g][2 * d * d + d: 2 * d * d + 2 * d] - ref["mu5"]).max() < 2e-6


# ------------------------------------------------------------------ fits
def invariants(p, d):
    """Quantities that do not depend on eigenvector signs or rotations in equal eigenvalues."""
    return {
        "eigA": np.sort(np.linalg.eigvalsh(p["A"])),
        "logD": np.array([p["logD"]]),
        "objective": np.array([p["objective"]]),
        "B1tB1": p["B1"].T @ p["B1"], "B2tB2": p["B2"].T @ p["B2"], "B1tB2": p["B1"].T @ p["B2"],
        "C1": p["C1"], "C2": p["C2"],
        "B1tAB1": p["B1"].T @ p["A"] @ p["B1"],
    }


def assert_fit_close(got, ref, d, tol):
    gi, ri = invariants(got, d), invariants(ref, d)
    for k in ri:
        scale = max(np.abs(ri[k]).max(), 1e-30)
        assert np.abs(gi[k] - ri[k]).max() <= tol * scale, (k, np.abs(gi[k] - ri[k]).max() / scale)


@pytest.mark.parametrize("variant", ["posrf", "gerf", "saderf", "aderf", "sderf"])
@pytest.mark.parametrize("d", [16, 64, 128])
def test_fit_from_exact_statistics(ctx, variant, d):
    """The fit kernel alone: statistics computed by the checker in fp64, uploaded, fitted on
    the GPU; invariants agree to 1e-9 and the blob satisfies Theorem 4.1's conditions."""
    rng = np.random.default_rng(100 + d)
    G, L = 3, 4 * d
    sl = fb.stats_doubles(d)
    blob = np.zeros((G, sl))
    refs = []
    for g in range(G):
        X = rng.standard_normal((L, d)) * rng.uniform(0.5, 1.5, d) / d ** 0.25 + 0.05 * g
        Y = rng.standard_normal((L, d)) * rng.uniform(0.5, 1.5, d) / d ** 0.25 - 0.03
        st = fs.set_statistics(X, Y)
        blob[g, : d * d] = st["M1"].ravel()
        blob[g, d * d: 2 * d * d] = st["M2"].ravel()
        blob[g, 2 * d * d: 2 * d * d + d] = st["mu4"]
        blob[g, 2 * d * d + d: 2 * d * d + 2 * d] = st["mu5"]
        refs.append(fs.FITS[variant](st))
    pr = ctx.fsharp_fit_params(torch.from_numpy(blob).cuda(), d, variant)
    assert ctx.status() == 0
    pr = pr.cpu().numpy()
    I = np.eye(d)
    for g in range(G):
        p = fb.unpack_params(pr[g], d)
        assert_fit_close(p, refs[g], d, 1e-9)
        Sinv = np.linalg.inv(I - 4 * p["A"])
        assert np.abs(p["B1"].T @ Sinv @ p["B2"] - I).max() < 1e-9
        assert np.abs(p["C1"] + 0.5 * p["B1"].T @ Sinv @ p["B1"]).max() < 1e-9 * max(1, np.abs(p["C1"]).max())
        if variant == "sderf":
            a = np.diag(p["A"])
            assert np.all(np.diff(a) >= -1e-15)          # eigenvalues of N non-ascending


@pytest.mark.parametrize("variant", ["sderf", "aderf"])
@pytest.mark.parametrize("d", [16, 32, 64])
@pytest.mark.parametrize("case", ["all_equal", "clusters", "near_clusters", "two_equal_blocks"])
def test_fit_with_repeated_eigenvalues(ctx, variant, d, case):
    """Spectra on which an eigenvector-per-eigenvalue solver has no unique answer (eigenvalues equal or equal to
    rounding, a matrix that splits into blocks with the same spectrum): the fit must still give the invariants
    of the closed forms, whichever of its eigensolvers ends up doing the work."""
    rng = np.random.default_rng(7 * d + len(case))
    Qm, _ = np.linalg.qr(rng.standard_normal((d, d)))
    if case == "all_equal":
        M1 = 0.3 * np.eye(d)
    elif case in ("clusters", "near_clusters"):
        lam = np.repeat(np.linspace(0.1, 0.5, 8), d // 8)
        M1 = (Qm * lam) @ Qm.T
        if case == "near_clusters":
            E = rng.standard_normal((d, d))
            M1 = M1 + 1e-11 * (E + E.T)
    else:
        h = d // 2
        Bk = rng.standard_normal((h, h))
        Bk = Bk @ Bk.T / h + 0.1 * np.eye(h)
        M1 = np.zeros((d, d))
        M1[:h, :h] = Bk
        M1[h:, h:] = Bk
    M1 = 0.5 * (M1 + M1.T)
    M2 = 0.5 * M1 + 0.1 * np.eye(d)
    mu4 = np.zeros(d) if case != "near_clusters" else 1e-3 * rng.standard_normal(d)
    mu5 = np.zeros(d)
    st = {"M1": M1, "M2": M2, "mu4": mu4, "mu5": mu5, "mu3": float(mu4 @ mu5) / d, "d": d}
    ref = fs.FITS[variant](st)
    blob = np.concatenate([M1.ravel(), M2.ravel(), mu4, mu5])[None, :]
    pr = ctx.fsharp_fit_params(torch.from_numpy(blob).cuda(), d, variant)
    assert ctx.status() == 0
    p = fb.unpack_params(pr.cpu().numpy()[0], d)
    assert_fit_close(p, ref, d, 1e-8)
    I = np.eye(d)
    Sinv = np.linalg.inv(I - 4 * p["A"])
    assert np.abs(p["B1"].T @ Sinv @ p["B2"] - I).max() < 1e-9


@pytest.mark.parametrize("w", small_cases()[:5], ids=lambda w: w.name)
def test_stats_then_fit_end_to_end(ctx, w):
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    for variant in ("sderf", "aderf", "gerf", "saderf"):
        _, pr = gpu_fit(ctx, dQ, dK, w.d, variant)
        pr = pr.cpu().numpy()
        for b in range(w.B):
            for h in range(w.H):
                ref = fs.fit_params(Q[b, h], K[b, h], variant)
                assert_fit_close(fb.unpack_params(pr[b * w.H + h], w.d), ref, w.d, FIT_TOL)


# ------------------------------------------------------------------ featurize
@pytest.mark.parametrize("w", [small_cases()[0], small_cases()[1], small_cases()[2], small_cases()[4]], ids=lambda w: w.name)
@pytest.mark.parametrize("stab", [fb.STAB_NONE, fb.STAB_ROW, fb.STAB_GROUP])
@pytest.mark.parametrize("impl", [fb.IMPL_SIMT, fb.IMPL_AUTO])
def test_featurize_matches_definition(ctx, w, stab, impl):
    """Features element by element against the definition (Section 4 with Section 2.1's M^-1/2).  With IMPL_AUTO the
    bf16, d = 64, M = 256 cases with a row shift or none take the tensor-core kernel, whose arithmetic (fp16 image of
    W, per-feature term inside the MMA, exponentials shared between two pipes) is that of the attention kernels:
    its features are held to the bf16 tolerance, the fp32 kernels to 2e-4."""
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    prh = pr.cpu().numpy()
    tensor = impl == fb.IMPL_AUTO and w.dtype == "bf16" and w.d == 64 and w.M == 256 and stab != fb.STAB_GROUP
    ctx.set_impl(impl)
    try:
        for side, X, dX in ((1, Q, dQ), (2, K, dK)):
            n0 = ctx.launch_count()
            phi, ls = ctx.fsharp_featurize(dX, dOm, pr, side, stab=stab)
            assert ctx.status() == 0
            assert ctx.launch_count() - n0 == (3 if tensor else (5 if stab == fb.STAB_GROUP else 4))
            phi = host(phi)
            for b in range(w.B):
                for h in range(w.H):
                    p = fb.unpack_params(prh[b * w.H + h], w.d)
                    ref = fs.derf_log_features(X[b, h], Om, p["A"], p[f"B{side}"], p[f"C{side}"], p["logD"])
                    if stab == fb.STAB_ROW:
                        shift = host(ls)[b, h][:, None]
                        assert phi[b, h].max() <= 1.0 + 1e-6
                    elif stab == fb.STAB_GROUP:
                        shift = host(ls)[b, h]
                        assert abs(shift - ref.max()) < 1e-4 * max(1.0, abs(ref.max()))   # the exact maximum
                    else:
                        shift = 0.0
                    got = phi[b, h]
                    expect = np.exp(ref - shift)
                    big = expect > 1e-30                                # below that fp32 has flushed
                    tol = TOL["bf16"] if tensor else 2e-4
                    assert np.max(np.abs(got[big] / expect[big] - 1)) < tol
    finally:
        ctx.set_impl(fb.IMPL_AUTO)


def test_exponents_tensor_core_kernel_d128(ctx):
    """bf16 tokens with d = 128 take the tensor-core kernel for the exponents' product (W as a bf16 value and its
    remainder): a ragged tail, three feature blocks, [B, L, H, d] storage, parameters pooled per head, a query / key
    scale; element by element against the definition, and against the fp32 kernels."""
    w = W["cfg5"].scaled(B=2, H=3, L=300, M=384, outlier_frac=0.05)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    s = 0.9
    st = ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD, qk_scale=s)
    pr = ctx.fsharp_fit_params(st, w.d, "aderf")
    prh = pr.cpu().numpy()
    tr = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    for side, X, dX in ((1, Q, tr(dQ)), (2, K, tr(dK))):
        phi, ls = ctx.fsharp_featurize(dX, dOm, pr, side, pool=fb.POOL_PER_HEAD, qk_scale=s, stab=fb.STAB_ROW)
        ctx.set_impl(fb.IMPL_SIMT)
        try:
            phi32, ls32 = ctx.fsharp_featurize(dX, dOm, pr, side, pool=fb.POOL_PER_HEAD, qk_scale=s, stab=fb.STAB_ROW)
        finally:
            ctx.set_impl(fb.IMPL_AUTO)
        assert ctx.status() == 0
        assert (ls - ls32).abs().max().item() < 2e-4 and (phi - phi32).abs().max().item() < 2e-4
        phi, ls = host(phi), host(ls)
        for b in range(w.B):
            for h in range(w.H):
                p = fb.unpack_params(prh[h], w.d)
                ref = fs.derf_log_features(s * X[b, h], Om, p["A"], p[f"B{side}"], p[f"C{side}"], p["logD"])
                expect = np.exp(ref - ls[b, h][:, None])
                big = expect > 1e-30
                assert np.max(np.abs(phi[b, h][big] / expect[big] - 1)) < 2e-4
                assert np.max(np.abs(ls[b, h] - ref.max(axis=1))) < 2e-4 * max(1.0, np.abs(ref).max())


# ------------------------------------------------------------------ attend
@pytest.mark.parametrize("w", small_cases(), ids=lambda w: f"{w.name}-L{w.L}-{w.variant}")
@pytest.mark.parametrize("impl", [fb.IMPL_SIMT, fb.IMPL_AUTO])
def test_attend_small_full_parity(ctx, w, impl):
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    ctx.set_impl(impl)
    try:
        Y = ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=w.causal, chunk=w.chunk)
        assert ctx.status() == 0
    finally:
        ctx.set_impl(fb.IMPL_AUTO)
    Y = host(Y)
    prh = pr.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            ref = oracle_unit(Q, K, V, Om, prh[b * w.H + h], w.d, b, h, w.causal)
            assert rel_err(Y[b, h], ref) < TOL[w.dtype], (b, h)
            # element by element too, where the reference is not near zero
            worst, median = elem_err(Y[b, h], ref, 0.1)
            assert worst < ELEM_TOL[w.dtype][0] and median < ELEM_TOL[w.dtype][1], (b, h, worst, median)
    if w.causal:
        assert np.abs(Y[:, :, 0] - V[:, :, 0]).max() < (1e-5 if w.dtype == "f32" else 1e-2)


def test_attend_properties(ctx):
    w = W["cfg2"].scaled(B=1, H=3, L=384)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    ones = torch.ones_like(dV)
    Y1 = host(ctx.fsharp_attend(dQ, dK, ones, dOm, pr))
    assert np.abs(Y1 - 1).max() < 1e-2                      # right stochastic: V = 1 gives Y = 1
    Y = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr))
    perm = torch.randperm(w.L, generator=torch.Generator().manual_seed(1)).cuda()
    Yp = host(ctx.fsharp_attend(dQ, dK[:, :, perm].contiguous(), dV[:, :, perm].contiguous(), dOm, pr))
    assert np.abs(Y - Yp).max() < 2e-2                      # key order does not matter
    # causal: outputs before position t do not depend on tokens from t on; chunk size is immaterial
    wc = W["cfg3"].scaled(B=1, H=2, L=512)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(wc)
    _, pr = gpu_fit(ctx, dQ, dK, wc.d, wc.variant)
    Ya = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128))
    dK2, dV2 = dK.clone(), dV.clone()
    dK2[:, :, 300:] *= 1.5
    dV2[:, :, 300:] += 1.0
    Yb = host(ctx.fsharp_attend(dQ, dK2, dV2, dOm, pr, causal=True, chunk=128))
    # (the keys' shifts are taken over a chunk or the whole sequence, so the rounding may differ:
    # one bf16 unit in the last place of an output below 4)
    assert np.abs(Ya[:, :, :300] - Yb[:, :, :300]).max() <= 2.0 ** -6
    assert np.abs(Ya[:, :, 300:] - Yb[:, :, 300:]).max() > 0.1
    for ch in (64, 256):
        Yc = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=ch))
        assert rel_err(Yc, Ya) < 1e-2
    assert ctx.status() == 0


@pytest.mark.parametrize("stress", ["keys_ramp_up", "keys_ramp_down", "all_scaled"])
def test_bidirectional_tensor_core_path_wide_dynamic_range(ctx, stress):
    """Keys whose size changes threefold along the sequence (or queries and keys scaled 2.5x) spread the
    feature exponents over far more than fp16's range; the tensor-core kernels must still agree with
    the checker (per-feature scales of the contracted state, joined to the query logits)."""
    for variant in ("sderf", "aderf"):
        w = W["cfg3b"].scaled(B=1, H=2, L=896, variant=variant)
        Q, K, V = wl.make_qkv(w)
        Om = wl.make_omega(w)
        t = np.arange(w.L, dtype=np.float64) / w.L
        if stress == "all_scaled":
            Q, K = wl.bf16_round(Q * 2.5), wl.bf16_round(K * 2.5)
        else:
            gain = 1.0 + 2.0 * t if stress == "keys_ramp_up" else 3.0 - 2.0 * t
            K = wl.bf16_round(K * gain[None, None, :, None])
        dQ, dK, dV, dOm = dev(Q, "bf16"), dev(K, "bf16"), dev(V, "bf16"), dev(Om)
        _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
        Y = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr))
        assert ctx.status() == 0
        prh = pr.cpu().numpy()
        for h in range(w.H):
            ref = oracle_unit(Q, K, V, Om, prh[h], w.d, 0, h, False)
            assert rel_err(Y[0, h], ref) < TOL["bf16"], (variant, h)


@pytest.mark.parametrize("ramp", ["up", "down", "flat"])
def test_causal_tensor_core_path_scales_across_chunks(ctx, ramp):
    """bf16, d = dv = 64, M = 256, chunk 128 takes the tensor-core causal kernels.  Keys that grow
    (or shrink) along the sequence move the chunks' shifts far apart, which exercises the scale that
    joins the prefix term and the in-chunk term; the layout is [B, L, H, d] storage viewed as [B, H, L, d]."""
    w = W["cfg3"].scaled(B=2, H=2, L=896, variant="sderf")
    Q, K, V = wl.make_qkv(w)
    Om = wl.make_omega(w)
    t = np.arange(w.L, dtype=np.float64) / w.L
    gain = {"up": 1.0 + 2.0 * t, "down": 3.0 - 2.0 * t, "flat": np.ones_like(t)}[ramp]
    K = wl.bf16_round(K * gain[None, None, :, None])
    dQ, dK, dV, dOm = dev(Q, "bf16"), dev(K, "bf16"), dev(V, "bf16"), dev(Om)
    strided = lambda x: x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    dQ, dK, dV = strided(dQ), strided(dK), strided(dV)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    Y = ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128)
    assert ctx.status() == 0
    ctx.set_impl(fb.IMPL_SIMT)
    try:
        Ys = ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128)
    finally:
        ctx.set_impl(fb.IMPL_AUTO)
    Y, Ys = host(Y), host(Ys)
    prh = pr.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            ref = oracle_unit(Q, K, V, Om, prh[b * w.H + h], w.d, b, h, True)
            assert rel_err(Y[b, h], ref) < TOL["bf16"], (b, h)
            assert rel_err(Ys[b, h], ref) < TOL["bf16"], (b, h)
    assert np.abs(Y[:, :, 0] - V[:, :, 0]).max() < 1e-2          # the first query sees only the first key


@pytest.mark.gpu
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("slices", [(512, 512, 512), (600, 424, 512), (1280,), (130, 1150)])
def test_sequence_parallel_key_states(ctx, causal, slices):
    """Sequence parallelism (the token axis cut into contiguous slices, one per rank): every slice's keys are reduced
    to a key state, the states are handed round, and every slice's queries are finished from the states they may see.
    The ranks are emulated one after the other on this device (their kernels do not wait on one another); the result
    must match the definition on the whole sequence, and the single call on the whole sequence."""
    from paper_2302_00787_b200 import sharding
    L = sum(slices)
    w = W["cfg3"].scaled(B=1, H=3, L=L, variant="aderf")
    Q, K, V = wl.make_qkv(w)
    Om = wl.make_omega(w)
    t = np.arange(L, dtype=np.float64) / L
    K = wl.bf16_round(K * (1.0 + 1.5 * t)[None, None, :, None])       # the slices' shifts differ
    dQ, dK, dV, dOm = dev(Q, "bf16"), dev(K, "bf16"), dev(V, "bf16"), dev(Om)
    # per-slice statistics combined with the slice lengths as weights = statistics of the whole sequence
    off = np.concatenate([[0], np.cumsum(slices)])
    cut = lambda x, r: x[:, :, off[r]:off[r + 1]].contiguous()
    st_all = ctx.fsharp_stats(dQ, dK)
    st = sum(ctx.fsharp_stats(cut(dQ, r), cut(dK, r)) * float(n) for r, n in enumerate(slices)) / float(L)
    assert float((st - st_all).abs().max()) <= 2e-6 * float(st_all.abs().max())    # (fp32 products per tile, fp64 sums)
    pr = ctx.fsharp_fit_params(st, w.d, w.variant)
    gathered = [ctx.fsharp_attend_key_state(cut(dK, r), cut(dV, r), dOm, pr) for r in range(len(slices))]
    Y = torch.empty(w.B, w.H, L, w.dv, dtype=dQ.dtype, device="cuda")
    for r in range(len(slices)):
        states, shifts = sharding.select_states(gathered, r, causal)
        Y[:, :, off[r]:off[r + 1]] = ctx.fsharp_attend_with_state(cut(dQ, r), cut(dK, r), cut(dV, r), dOm, pr, states, shifts,
                                                                  causal=causal)
    assert ctx.status() == 0
    Y1 = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=causal, chunk=128)) if L % 128 == 0 else None
    Y = host(Y)
    prh = pr.cpu().numpy()
    for h in range(w.H):
        ref = oracle_unit(Q, K, V, Om, prh[h], w.d, 0, h, causal)
        assert rel_err(Y[0, h], ref) < TOL["bf16"], h
        if Y1 is not None:                   # two results that are each within the tolerance of the definition
            assert rel_err(Y[0, h], Y1[0, h]) < 2 * TOL["bf16"], h


@pytest.mark.gpu
def test_sequence_parallel_argument_checks(ctx):
    w = W["cfg3"].scaled(B=1, H=1, L=256, variant="sderf")
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    state, shifts = ctx.fsharp_attend_key_state(dK, dV, dOm, pr)
    assert state.shape[0] == 1 and state.shape[2:] == (80, 256) and shifts.shape == (1, state.shape[1], 2)
    with pytest.raises(fb.FsharpError) as e:            # bidirectional: every key must be behind a state
        ctx.fsharp_attend_with_state(dQ, dK, dV, dOm, pr, None, None, causal=False)
    assert e.value.code == -2
    with pytest.raises(fb.FsharpError) as e:            # the tensor-core kernels' shape only
        ctx.fsharp_attend_key_state(dK.float(), dV.float(), dOm, pr)
    assert e.value.code == -2
    with pytest.raises(ValueError):
        ctx.fsharp_attend_with_state(dQ, dK, dV, dOm, pr, state[:, :, :40], shifts, causal=True)
    many = state[:, :1].expand(1, 65, 80, 256).contiguous()                      # more states than one launch merges
    with pytest.raises(fb.FsharpError) as e:
        ctx.fsharp_attend_with_state(dQ, None, None, dOm, pr, many, shifts[:, :1].expand(1, 65, 2).contiguous(), causal=False)
    assert e.value.code == -10
    # the same states twice = every key counted twice: numerator and normaliser double, the output does not change
    twice = (torch.cat([state, state], dim=1).contiguous(), torch.cat([shifts, shifts], dim=1).contiguous())
    Ya = host(ctx.fsharp_attend_with_state(dQ, None, None, dOm, pr, state, shifts, causal=False))
    Yb = host(ctx.fsharp_attend_with_state(dQ, None, None, dOm, pr, twice[0], twice[1], causal=False))
    assert np.abs(Ya - Yb).max() <= 2.0 ** -7 * np.abs(Ya).max()
    assert rel_err(Ya, host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr))) < 2 * TOL["bf16"]
    # strided tensors ([B, L, H, d] storage) and one parameter group per head
    tr = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    st_h = ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD)
    pr_h = ctx.fsharp_fit_params(st_h, w.d, w.variant)
    s2, h2 = ctx.fsharp_attend_key_state(tr(dK), tr(dV), dOm, pr_h, pool=fb.POOL_PER_HEAD)
    Yc = host(ctx.fsharp_attend_with_state(tr(dQ), None, None, dOm, pr_h, s2, h2, causal=False, pool=fb.POOL_PER_HEAD))
    assert rel_err(Yc, host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr_h, pool=fb.POOL_PER_HEAD))) < 2 * TOL["bf16"]
    # causal with nothing before it is the plain causal call
    Y0 = host(ctx.fsharp_attend_with_state(dQ, dK, dV, dOm, pr, None, None, causal=True))
    Y1 = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128))
    assert np.array_equal(Y0, Y1)
    assert ctx.status() == 0


def test_attend_strided_layout_per_head_omega_and_pooling(ctx):
    w = W["cfg2"].scaled(B=2, H=3, L=256)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    OmH = np.stack([wl.orthogonal_omega(w.M, w.d, 77 + h) for h in range(w.H)])
    dOmH = dev(OmH)
    st = ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD)
    pr = ctx.fsharp_fit_params(st, w.d, "sderf")
    tr = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    out = torch.empty(w.B, w.L, w.H, w.dv, dtype=dQ.dtype, device="cuda").permute(0, 2, 1, 3)
    Y = ctx.fsharp_attend(tr(dQ), tr(dK), tr(dV), dOmH, pr, pool=fb.POOL_PER_HEAD, out=out)
    assert ctx.status() == 0
    Y = host(Y)
    prh = pr.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            p = fb.unpack_params(prh[h], w.d)
            ref = fs.favor_sharp_attention(Q[b, h], K[b, h], V[b, h], OmH[h], p)
            assert rel_err(Y[b, h], ref) < TOL["bf16"]


@pytest.mark.parametrize("chunk,M", [(128, 256), (256, 384), (64, 512)])
def test_causal_d128_chain_of_tensor_core_kernels(ctx, chunk, M):
    """bf16, d = dv = 128 has no fused kernel: exponents, in-chunk scores, per-chunk key-side sums and the query side
    each run on the tensor cores (chunk 64 leaves the last three to the fp32 kernels).  [B, L, H, *] storage,
    per-head Omega, parameters pooled per head, several chunks, a query / key scale; against the definition, unit by
    unit, and against the fp32 kernels."""
    w = W["cfg5"].scaled(B=2, H=2, L=768, M=M, chunk=chunk, outlier_frac=0.05)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    OmH = np.stack([wl.orthogonal_omega(w.M, w.d, 31 + h) for h in range(w.H)])
    s = 0.95
    st = ctx.fsharp_stats(dQ, dK, pool=fb.POOL_PER_HEAD, qk_scale=s)
    pr = ctx.fsharp_fit_params(st, w.d, "sderf")
    tr = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    out = torch.empty(w.B, w.L, w.H, w.dv, dtype=dQ.dtype, device="cuda").permute(0, 2, 1, 3)
    n0 = ctx.launch_count()
    Y = ctx.fsharp_attend(tr(dQ), tr(dK), tr(dV), dev(OmH), pr, causal=True, chunk=chunk, pool=fb.POOL_PER_HEAD, qk_scale=s, out=out)
    launches = ctx.launch_count() - n0
    ctx.set_impl(fb.IMPL_SIMT)
    try:
        Y32 = ctx.fsharp_attend(tr(dQ), tr(dK), tr(dV), dev(OmH), pr, causal=True, chunk=chunk, pool=fb.POOL_PER_HEAD, qk_scale=s)
    finally:
        ctx.set_impl(fb.IMPL_AUTO)
    assert ctx.status() == 0 and launches == 12        # prep; 4 + 3 feature kernels; sums, scan, scores, query side
    Y, Y32 = host(Y), host(Y32)
    prh = pr.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            p = fb.unpack_params(prh[h], w.d)
            ref = fs.favor_sharp_attention(Q[b, h], K[b, h], V[b, h], OmH[h], p, causal=True, qk_scale=s)
            assert rel_err(Y[b, h], ref) < TOL["bf16"], (b, h, rel_err(Y[b, h], ref))
            assert rel_err(Y32[b, h], ref) < TOL["bf16"]
            assert rel_err(Y[b, h], Y32[b, h]) < TOL["bf16"]
    assert np.abs(Y[:, :, 0] - V[:, :, 0]).max() < 1e-2        # the first token attends to itself only


def test_qk_scale_is_applied(ctx):
    w = W["cfg1"]
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    s = w.d ** -0.25
    st = ctx.fsharp_stats(dQ, dK, qk_scale=s)
    pr = ctx.fsharp_fit_params(st, w.d, "sderf")
    Y = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, qk_scale=s))
    p = fb.unpack_params(pr.cpu().numpy()[0], w.d)
    ref = fs.favor_sharp_attention(Q[0, 0], K[0, 0], V[0, 0], Om, p, qk_scale=s)
    assert rel_err(Y[0, 0], ref) < TOL["f32"]
    refp = fs.fit_params(s * Q[0, 0].astype(np.float64), s * K[0, 0].astype(np.float64), "sderf")
    assert abs(p["objective"] - refp["objective"]) < FIT_TOL * abs(refp["objective"])


def test_forward_host_matches_device_path(ctx):
    w = W["cfg3"].scaled(B=1, H=2, L=256)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    Yd = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128))
    pin = lambda t: t.cpu().contiguous().pin_memory()
    Yh = ctx.fsharp_forward_host(pin(dQ), pin(dK), pin(dV), pin(dOm), w.variant, causal=True, chunk=128)
    assert np.abs(host(Yh) - Yd).max() < 2e-2
    assert rel_err(host(Yh)[0, 0], oracle_unit(Q, K, V, Om, pr.cpu().numpy()[0], w.d, 0, 0, True)) < TOL["bf16"]


# ------------------------------------------------------------------ edge cases and errors
def test_empty_and_degenerate_inputs(ctx):
    d, M = 16, 32
    Om = dev(wl.iid_omega(M, d, 1))
    pr = torch.zeros(1, fb.params_doubles(d), dtype=torch.float64, device="cuda")
    e = torch.empty(1, 1, 0, d, device="cuda")
    assert ctx.fsharp_attend(e, e, e, Om, pr).shape == (1, 1, 0, d)            # no query: nothing to do
    e0 = torch.empty(0, 1, 8, d, device="cuda")
    assert ctx.fsharp_stats(e0, e0).shape[0] == 0
    # single token: Y = V exactly (one key carries all the weight)
    w = W["cfg1"].scaled(L=1)
    (Q, K, V, Om1), (dQ, dK, dV, dOm) = upload(w)
    st = ctx.fsharp_stats(dQ, dK)
    prg = ctx.fsharp_fit_params(st, w.d, "gerf")
    Y = host(ctx.fsharp_attend(dQ, dK, dV, dOm, prg))
    assert np.abs(Y - V).max() < 1e-5
    assert ctx.status() == 0


def test_error_codes(ctx):
    w = W["cfg1"].scaled(L=64)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, "sderf")

    def code(fn):
        with pytest.raises(fb.FsharpError) as ei:
            fn()
        return ei.value.code

    assert code(lambda: ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=48)) == -2     # chunk size
    assert code(lambda: ctx.fsharp_attend(dQ[:, :, :40].contiguous(), dK[:, :, :40].contiguous(),
                                          dV[:, :, :40].contiguous(), dOm, pr, causal=True, chunk=64)) == -2
    bad = torch.empty(1, 1, 64, 24, device="cuda")
    assert code(lambda: ctx.fsharp_stats(bad, bad)) == -2                                         # d = 24
    flat = torch.empty(64 * 16 + 1, device="cuda")[1:].view(1, 1, 64, 16)
    assert code(lambda: ctx.fsharp_stats(flat, flat)) == -3                                       # misaligned
    assert code(lambda: ctx.fsharp_attend(dQ, dK[:, :, :0], dV[:, :, :0], dOm, pr)) == -2         # no keys
    # fp32 causal: (batch, head, chunk) is a grid coordinate of at most 65535; refused as a shape, before any launch
    wide = dQ[:, :1, :1].expand(1, 1024, 4096, 16)
    n0 = ctx.launch_count()
    assert code(lambda: ctx.fsharp_attend(wide, wide, wide, dOm, pr, causal=True, chunk=64)) == -2
    assert ctx.launch_count() == n0
    lib = fb.load_library()
    assert lib.fsharp_fit_params(ctx._h, None, 1, 16, 4, 0.0, pr.data_ptr()) == -1
    assert lib.fsharp_fit_params(ctx._h, pr.data_ptr(), 1, 16, 9, 0.0, pr.data_ptr()) == -1
    assert ctx.status() == 0


def test_device_detected_conditions(ctx):
    w = W["cfg1"].scaled(L=64)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    dQn = dQ.clone()
    dQn[0, 0, 3, 5] = float("nan")
    ctx.fsharp_stats(dQn, dK)
    assert ctx.status() == -7                      # non-finite input
    assert ctx.status() == 0                       # reading clears it
    dQz = dQ.clone()
    dQz[..., 2] = 0.0                              # a zero column makes M1 singular
    st = ctx.fsharp_stats(dQz, dK)
    ctx.fsharp_fit_params(st, w.d, "aderf")
    assert ctx.status() == -6
    pr = ctx.fsharp_fit_params(st, w.d, "aderf", ridge=1e-3)     # the ridge repairs it
    assert ctx.status() == 0
    assert torch.isfinite(pr).all()


# ------------------------------------------------------------------ pairs
@pytest.mark.parametrize("variant", ["aderf", "sderf", "gerf", "posrf"])
def test_pair_estimates_and_closed_form_variance(ctx, variant):
    npairs, d, M, R = 1000, 64, 64, 3
    X, Y = wl.make_pairs(npairs, d)
    Om = np.stack([wl.orthogonal_omega(M, d, 4000 + r) for r in range(R)])
    dX, dY = dev(X), dev(Y)
    st = ctx.fsharp_stats(dX.view(1, 1, npairs, d), dY.view(1, 1, npairs, d))
    pr = ctx.fsharp_fit_params(st, d, variant)
    est, var = ctx.fsharp_pair_estimate(dX, dY, dev(Om), pr)
    assert ctx.status() == 0
    p = fb.unpack_params(pr.cpu().numpy()[0], d)
    for r in range(R):
        ref = fs.pair_estimate(X, Y, Om[r], p)
        assert np.max(np.abs(host(est[r]) / ref - 1)) < 1e-4
    sel = np.arange(0, npairs, 37)
    refv = fs.pair_closed_form_variance(X[sel], Y[sel], p, M)
    assert np.max(np.abs(var.cpu().numpy()[sel] / refv - 1)) < 1e-8


# ------------------------------------------------------------------ several steps in flight
@pytest.mark.parametrize("alpha", [0.0, -0.5])
@pytest.mark.parametrize("w", [W["cfg1"], W["cfg2"].scaled(B=1, H=2, L=300), W["cfg3b"].scaled(B=2, H=1, L=200)],
                         ids=lambda w: f"{w.name}-{w.variant}")
def test_unnormalised_operator_matches_definition(ctx, w, alpha):
    """Khat^(alpha) C of Sections 2.1 / 2.3 (alpha = 0: softmax kernel, alpha = -1/2: Gaussian kernel) against the
    checker on the same Omega and the same parameter blob, relative to the largest output of the (batch, head);
    the sets X and Y have different sizes."""
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    Lq = w.L - 37
    out = ctx.fsharp_kernel_apply(dQ[:, :, :Lq].contiguous(), dK, dV, dOm, pr, alpha=alpha)
    assert ctx.status() == 0
    out = host(out)
    prh = pr.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            p = fb.unpack_params(prh[b * w.H + h], w.d)
            ref = fs.kernel_apply(Q[b, h, :Lq], K[b, h], V[b, h], Om, p, alpha)
            assert rel_err(out[b, h], ref) < TOL[w.dtype], (b, h)
    with pytest.raises(fb.FsharpError) as ei:
        ctx.fsharp_kernel_apply(dQ, dK[:, :, :0], dV[:, :, :0], dOm, pr, alpha=alpha)
    assert ei.value.code == -2


def test_bounded_wait_runs_out_and_the_context_stays_usable(ctx):
    """Every device-side wait is bounded.  The self-test kernel waits 2 ms on a barrier that nothing completes: the
    wait gives up, the kernel returns, the status word reports the time-out, and the next call works."""
    w = W["cfg3"].scaled(B=1, H=1, L=256)
    (Q, K, V, Om), (dQ, dK, dV, dOm) = upload(w)
    _, pr = gpu_fit(ctx, dQ, dK, w.d, w.variant)
    ctx.selftest_bounded_wait(2000)
    assert ctx.status() == -8                     # FSHARP_E_TIMEOUT, latched once ...
    assert ctx.status() == 0                      # ... and cleared by the read
    Y = host(ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=True, chunk=128))
    assert ctx.status() == 0
    ref = oracle_unit(Q, K, V, Om, pr.cpu().numpy()[0], w.d, 0, 0, True)
    assert rel_err(Y[0, 0], ref) < TOL["bf16"]
    with pytest.raises(fb.FsharpError):
        ctx.selftest_bounded_wait(0)


def test_debug_build_index_checks_stay_silent():
    """The build with -DFSHARP_DEBUG checks tile, shared-memory and tensor-memory indices inside the tensor-core
    kernels and latches an error instead of faulting.  Run small cases of every tensor-core kernel through it in a
    process of its own (another build of the same library): no check fires and the results are finite."""
    import subprocess, sys, os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    lib = os.path.join(root, "paper_2302_00787_b200", "lib", "libfsharp_debug.so")
    if not os.path.exists(lib):
        from paper_2302_00787_b200 import build as b
        b.build(debug=True)
    script = """
import torch
from paper_2302_00787_b200 import binding as fb, workloads as wl
assert fb.LIB_PATH.endswith('libfsharp_debug.so')
ctx = fb.Context(0)
for w in (wl.WORKLOADS['cfg2'].scaled(B=2, H=2, L=300), wl.WORKLOADS['cfg3'].scaled(B=1, H=3, L=1024),
          wl.WORKLOADS['cfg3b'].scaled(B=1, H=2, L=640), wl.WORKLOADS['cfg3'].scaled(B=1, H=150, L=640)):
    Q, K, V = wl.make_qkv(w); Om = wl.make_omega(w)
    dQ, dK, dV = (torch.from_numpy(a).cuda().to(torch.bfloat16) for a in (Q, K, V)); dOm = torch.from_numpy(Om).cuda()
    st = ctx.fsharp_stats(dQ, dK); pr = ctx.fsharp_fit_params(st, w.d, w.variant)
    Y = ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=w.causal, chunk=w.chunk)
    phi, ls = ctx.fsharp_featurize(dK, dOm, pr, 2, stab=fb.STAB_ROW)
    assert ctx.status() == 0, w
    assert torch.isfinite(Y.float()).all() and torch.isfinite(phi).all()
print('debug build ok')
"""
    env = dict(os.environ, FSHARP_LIB=lib, PYTHONPATH=root)
    r = subprocess.run([sys.executable, "-c", script], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout + r.stderr


def test_variance_study_batch_many_pairs_many_draws(ctx):
    """The variance-study batch at 2^16 pairs and 32 draws (a multi-wave grid for the estimates, the grid-stride
    loops of the per-pair variance and of the pooling): estimates on sampled pairs for every draw, closed-form
    variances on sampled pairs, and the two pooled relative variances, against the checker."""
    pw = wl.PAIR_WORKLOADS["cfg4"].scaled(npairs=2 ** 16)
    X, Y = wl.make_pairs(pw.npairs, pw.d, pw.seed)
    Om = wl.make_pair_omegas(pw)
    dX, dY, dOm = dev(X), dev(Y), dev(Om)
    st = ctx.fsharp_stats(dX.view(1, 1, pw.npairs, pw.d), dY.view(1, 1, pw.npairs, pw.d))
    rng = np.random.default_rng(5)
    sel = np.unique(np.concatenate([rng.integers(0, pw.npairs, 500), np.arange(pw.npairs - 70, pw.npairs), [0, 63, 64]]))
    dXs, dYs = dev(X[sel]), dev(Y[sel])
    for variant in pw.variants:
        pr = ctx.fsharp_fit_params(st, pw.d, variant)
        est, var, pooled = ctx.fsharp_pair_estimate(dX, dY, dOm, pr, want_pooled=True)
        assert ctx.status() == 0
        p = fb.unpack_params(pr.cpu().numpy()[0], pw.d)
        ref = np.stack([fs.pair_estimate(X[sel], Y[sel], Om[r], p) for r in range(pw.R)])
        assert np.max(np.abs(host(est)[:, sel] / ref - 1)) < 1e-4, variant
        vsel = sel[::4]
        refv = fs.pair_closed_form_variance(X[vsel], Y[vsel], p, pw.M)
        assert np.max(np.abs(var.cpu().numpy()[vsel] / refv - 1)) < 1e-8, variant
        # pooled numbers of the full batch: the reduction over all pairs of the per-pair quantities just checked
        K2 = torch.exp(2.0 * (dX.double() * dY.double()).sum(dim=1))
        emp_full = (est.double().var(dim=0, unbiased=True) / K2).mean().item()
        cf_full = (var / K2).mean().item()
        assert abs(pooled[0].item() / emp_full - 1) < 1e-9 and abs(pooled[1].item() / cf_full - 1) < 1e-9, variant
        # and on the sampled pairs alone, where the checker computes both numbers itself
        est_s, var_s, pooled_s = ctx.fsharp_pair_estimate(dXs, dYs, dOm, pr, want_pooled=True)
        emp_ref, cf_ref = fs.pair_pooled_relative_variance(ref, X[sel], Y[sel], fs.pair_closed_form_variance(X[sel], Y[sel], p, pw.M))
        assert abs(pooled_s[0].item() / emp_ref - 1) < 1e-3, variant      # fp32 estimates: their variance to 1e-3
        assert abs(pooled_s[1].item() / cf_ref - 1) < 1e-8, variant
    assert ctx.status() == 0


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_contexts_on_separate_streams_overlap_without_interference(ctx, name):
    """Three contexts, each with a stream, scratch block and outputs of its own, run whole steps
    (statistics, fit, attend) on different inputs at the same time, as the benchmark does.  With
    whole tiles (L a multiple of 128) the statistics kernel sums in a fixed order, so every result
    must equal, bit for bit, what one context computes for the same input on its own.  (With a
    ragged tail the statistics differ in the last bit from run to run, and Theorem 4.3's B, built
    on eigenvectors of nearly equal eigenvalues, then comes out as another of its many solutions:
    no run-to-run comparison of outputs is meaningful there.)  One result is also checked against
    the checker."""
    base = W[name].scaled(B=2, H=3, L=1024)
    n = 3
    inputs = [upload(base.scaled(seed=base.seed + 17 * i)) for i in range(n)]
    serial = []
    for (_, (dQ, dK, dV, dOm)) in inputs:
        _, pr = gpu_fit(ctx, dQ, dK, base.d, base.variant)
        serial.append((pr.clone(), ctx.fsharp_attend(dQ, dK, dV, dOm, pr, causal=base.causal, chunk=base.chunk).clone()))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(n)]
    ctxs = [fb.Context(0, stream=s) for s in streams]
    try:
        # every context writes into tensors of its own, allocated once (torch's allocator hands a freed block to
        # the next request at once, whatever stream still uses it)
        G = base.B * base.H
        sts = [torch.empty(G, fb.stats_doubles(base.d), dtype=torch.float64, device="cuda") for _ in range(n)]
        prs = [torch.empty(G, fb.params_doubles(base.d), dtype=torch.float64, device="cuda") for _ in range(n)]
        Ys = [torch.empty_like(serial[i][1]) for i in range(n)]
        torch.cuda.synchronize()
        for rep in range(4):                     # several rounds, so that kernels of different steps meet
            for i, (_, (dQ, dK, dV, dOm)) in enumerate(inputs):
                ctxs[i].fsharp_stats(dQ, dK, out=sts[i])
                ctxs[i].fsharp_fit_params(sts[i], base.d, base.variant, out=prs[i])
                ctxs[i].fsharp_attend(dQ, dK, dV, dOm, prs[i], causal=base.causal, chunk=base.chunk, out=Ys[i])
        torch.cuda.synchronize()
        for i in range(n):
            assert ctxs[i].status() == 0
            assert torch.equal(prs[i], serial[i][0]), f"parameters of step {i} differ when steps overlap"
            assert torch.equal(Ys[i], serial[i][1]), f"outputs of step {i} differ when steps overlap"
    finally:
        for c in ctxs:
            c.close()
    (Q, K, V, Om), _ = inputs[1]
    Y = host(Ys[1])
    blob = host(prs[1])
    for b in range(base.B):
        for h in range(base.H):
            ref = oracle_unit(Q, K, V, Om, blob[b * base.H + h], base.d, b, h, base.causal)
            assert rel_err(Y[b, h], ref) < TOL[base.dtype]
