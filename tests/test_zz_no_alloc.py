"""The no-allocation feature entry point (fsharp_featurize_static) against fsharp_featurize.

Collected last on purpose (file name): a run that stops at the first failure has by then
already run every other test.  The entry point exists for callers that cannot allocate device
memory at call time (foreign memory pools, allocator-free real-time loops, fully committed
HBM); it works out of a fixed array inside the loaded module, so this test also checks that
two calls in a row -- which share that array and find the previous call's contents in it --
both reproduce the allocating entry point."""
import numpy as np
import pytest
import torch

from oracle import favor_sharp as fs
from paper_2302_00787_b200 import binding as fb
from paper_2302_00787_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _inputs(w):
    Q, K, V = wl.make_qkv(w)
    Om = wl.make_omega(w)
    td = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    return (Q, K, Om), (torch.from_numpy(Q).cuda().to(td), torch.from_numpy(K).cuda().to(td), torch.from_numpy(Om).cuda())


def test_static_scratch_entry_point_matches_featurize_twice_in_a_row():
    ctx = fb.Context(0)
    cases = [(wl.WORKLOADS["cfg2"].scaled(B=1, H=2, L=300), 1, fb.STAB_ROW),
             (wl.WORKLOADS["cfg3"].scaled(B=1, H=2, L=256), 2, fb.STAB_GROUP)]
    for call, (w, side, stab) in enumerate(cases):   # two calls in a row on the shared scratch, different problems
        (Q, K, Om), (dQ, dK, dOm) = _inputs(w)
        X = dQ if side == 1 else dK
        st = ctx.fsharp_stats(dQ, dK)
        pr = ctx.fsharp_fit_params(st, w.d, w.variant)
        ctx.set_impl(fb.IMPL_SIMT)          # the entry point under test runs the fp32 kernels: compare like with like
        ref_phi, ref_ls = ctx.fsharp_featurize(X, dOm, pr, side, stab=stab)
        ctx.set_impl(fb.IMPL_AUTO)
        assert ctx.status() == 0
        phi = torch.full_like(ref_phi, float("nan"))
        ls = torch.full_like(ref_ls, float("nan"))
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]        # driver-level free bytes: moves only on a real allocation
        rc = fb.fsharp_featurize_static(X, dOm, pr, side, phi, ls, stab=stab, device_status=status)
        torch.cuda.synchronize()
        assert rc == 0
        if call > 0:      # the first call may load the module (and with it the fixed array) lazily
            assert torch.cuda.mem_get_info()[0] == free_before
        assert int(status.item()) == 0
        got, ref = phi.cpu().numpy().astype(np.float64), ref_phi.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        # same tolerance as the featurize parity test (relative, on entries fp32 has not flushed)
        big = ref > 1e-30
        assert np.max(np.abs(got[big] / ref[big] - 1)) < 2e-4
        assert np.max(np.abs(ls.cpu().numpy() - ref_ls.cpu().numpy())) < 1e-4
        # and against the fp64 checker itself, not only against the library's other entry point: the features of
        # one (batch, head) from the definition (Section 4 with Section 2.1's M^-1/2), on the same parameter blob
        p = fb.unpack_params(pr.cpu().numpy()[1], w.d)
        Xh = (Q if side == 1 else K)[0, 1]
        logf = fs.derf_log_features(Xh, Om, p["A"], p[f"B{side}"], p[f"C{side}"], p["logD"])
        shift = ls.cpu().numpy().astype(np.float64)[0, 1]
        expect = np.exp(logf - (shift[:, None] if stab == fb.STAB_ROW else shift))
        big = expect > 1e-30
        assert np.max(np.abs(got[0, 1][big] / expect[big] - 1)) < 2e-4
    ctx.close()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    assert fb.static_scratch_bytes() == 8 << 20
    # 64 groups x 2 sides x (1024*128 + ...) floats is far beyond 8 MiB: refused before any launch
    X = torch.zeros(1, 64, 16, 128, device="cuda")
    Om = torch.zeros(1024, 128, device="cuda")
    pr = torch.zeros(64, fb.params_doubles(128), dtype=torch.float64, device="cuda")
    phi = torch.zeros(1, 64, 16, 1024, device="cuda")
    ls = torch.zeros(1, 64, 16, device="cuda")
    assert fb.fsharp_featurize_static(X, Om, pr, 1, phi, ls) == -10
    assert "scratch" in fb.strerror(-10)
    assert fb.fsharp_featurize_static(X, Om, pr, 3, phi, ls) == -1          # bad side
    # the binding refuses outputs that the kernels would overrun
    with pytest.raises(ValueError):
        fb.fsharp_featurize_static(X, Om, pr, 1, phi[..., :512], ls)
    with pytest.raises(ValueError):
        fb.fsharp_featurize_static(X, Om, pr, 1, phi.double(), ls)
    with pytest.raises(ValueError):
        fb.fsharp_featurize_static(X, Om, pr, 1, phi, ls[:, :8], stab=fb.STAB_ROW)
