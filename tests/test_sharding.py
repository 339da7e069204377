"""Multi-GPU host logic on CPU: (batch, head) units are split over ranks with no data-path
collective; the only communication is the max / sum of scalars.  Two gloo ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2302_00787_b200 import sharding


def test_unit_partition_is_a_disjoint_cover():
    for n in (0, 1, 7, 48, 64):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(sharding.unit_partition(n, r, world))
            assert seen == list(range(n))
            sizes = [len(sharding.unit_partition(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.unit_partition(4, 2, 2)
    assert sharding.rank_seed(2000, 0) == 2000 and sharding.rank_seed(2000, 1) != 2000


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, lr, w = sharding.env_rank_world()
    import bench                                  # the benchmark's own rank set-up, as torchrun would start it
    assert bench.rank_setup(2) == (r, lr, w) == (rank, rank, world)

    class A:
        gpus, impl = 2, "native"
    assert bench.relaunch_if_needed(A) is False   # already under a launcher: no second one is started
    units = sharding.unit_partition(48, r, w)
    # each rank "times" its own share; the job's time is the slowest rank, its work the sum
    t = sharding.max_over_ranks(1.0 + 0.5 * r)
    n = sharding.sum_over_ranks(float(len(units)))
    dist.barrier()
    out.put((r, list(units), t, n))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_units_and_reduce_time():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] + res[1][1] == list(range(48))
    assert all(abs(t - 1.5) < 1e-12 and n == 48.0 for _, _, t, n in res)


def test_bench_starts_its_own_ranks_only_when_asked(monkeypatch):
    """`python bench.py --gpus N` outside a launcher re-executes itself under torch.distributed.run with N
    ranks on 127.0.0.1; with one GPU, under a launcher, or for the CPU reference arm it does not."""
    import bench

    class A:
        gpus, impl = 1, "native"
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    assert bench.relaunch_if_needed(A) is False
    A.gpus, A.impl = 4, "reference"
    assert bench.relaunch_if_needed(A) is False
    A.impl = "native"
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    with pytest.raises(SystemExit):
        bench.relaunch_if_needed(A)
    cmd = seen["cmd"]
    assert "torch.distributed.run" in cmd and "--nproc-per-node=4" in cmd and "127.0.0.1" in cmd
    assert bench.rank_setup(1) == (0, 0, 1)


# ---------------------------------------------------------------------------------------------
# Sequence parallelism on two gloo ranks.  The driver (sharding.sequence_parallel_forward) is the product's; the
# context it drives here is a stand-in that does every call in fp64 on the CPU with the checker's functions, so that
# what is tested is the exchange: token-weighted statistics, the order of the gathered key states, and which of them
# a rank's queries see.  Slices of unequal length.
# ---------------------------------------------------------------------------------------------
class _CheckerContext:
    def __init__(self):
        from oracle import favor_sharp as fo
        self.fo = fo

    def fsharp_stats(self, Q, K, qk_scale=1.0):
        B, H, _, d = Q.shape
        rows = []
        for b in range(B):
            for h in range(H):
                st = self.fo.set_statistics(qk_scale * Q[b, h].numpy(), qk_scale * K[b, h].numpy())
                rows.append(torch.from_numpy(__import__("numpy").concatenate(
                    [st["M1"].ravel(), st["M2"].ravel(), st["mu4"], st["mu5"]])))
        return torch.stack(rows)

    def fsharp_fit_params(self, stats, d, variant):
        out = []
        for row in stats.numpy():
            M1, M2 = row[:d * d].reshape(d, d), row[d * d:2 * d * d].reshape(d, d)
            mu4, mu5 = row[2 * d * d:2 * d * d + d], row[2 * d * d + d:]
            out.append(self.fo.FITS[variant]({"M1": M1, "M2": M2, "mu4": mu4, "mu5": mu5, "mu3": float(mu4 @ mu5) / d, "d": d}))
        return out

    def _S(self, K, Omega, p, qk_scale):
        return self.fo.derf_features(qk_scale * K.numpy(), Omega.numpy(), p["A"], p["B2"], p["C2"], p["logD"])

    def fsharp_attend_key_state(self, K, V, Omega, params, qk_scale=1.0):
        import numpy as np
        B, H, L, _ = K.shape
        blocks = []
        for b in range(B):
            for h in range(H):
                S = self._S(K[b, h], Omega, params[b * H + h], qk_scale)
                V1 = np.concatenate([V[b, h].numpy(), np.ones((L, 1))], axis=1)
                blocks.append(torch.from_numpy(S.T @ V1)[None])                 # one piece per call
        return torch.stack(blocks), torch.zeros(B * H, 1, 2, dtype=torch.float64)

    def fsharp_attend_with_state(self, Q, K, V, Omega, params, states, shifts, causal=False, qk_scale=1.0, out=None):
        import numpy as np
        B, H, L, _ = Q.shape
        Y = torch.empty(B, H, L, V.shape[-1], dtype=torch.float64)
        for b in range(B):
            for h in range(H):
                p = params[b * H + h]
                P = self.fo.derf_features(qk_scale * Q[b, h].numpy(), Omega.numpy(), p["A"], p["B1"], p["C1"], p["logD"])
                T = states[b * H + h].sum(dim=0).numpy() if states is not None else 0.0
                nd = P @ T if states is not None else np.zeros((L, V.shape[-1] + 1))
                if causal:
                    S = self._S(K[b, h], Omega, p, qk_scale)
                    V1 = np.concatenate([V[b, h].numpy(), np.ones((L, 1))], axis=1)
                    nd = nd + np.tril(P @ S.T) @ V1
                Y[b, h] = torch.from_numpy(nd[:, :-1] / nd[:, -1:])
        return Y


def _sp_worker(rank, world, port, out):
    import numpy as np
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import favor_sharp as fo
    rng = np.random.default_rng(5)
    B, H, d, dv, M = 1, 2, 8, 4, 16
    lens = [40, 24][:world]
    L = sum(lens)
    Q, K = rng.normal(size=(B, H, L, d)) / d ** 0.25, rng.normal(size=(B, H, L, d)) / d ** 0.25 + 0.1
    V, Om = rng.normal(size=(B, H, L, dv)), rng.normal(size=(M, d))
    lo = sum(lens[:rank])
    sl = lambda x: torch.from_numpy(np.ascontiguousarray(x[:, :, lo:lo + lens[rank]]))
    res = {}
    for causal in (False, True):
        Y = sharding.sequence_parallel_forward(_CheckerContext(), sl(Q), sl(K), sl(V), torch.from_numpy(Om), "sderf",
                                               causal=causal)
        err = 0.0
        for h in range(H):
            p = fo.fit_params(Q[0, h], K[0, h], "sderf")
            ref = fo.favor_sharp_attention(Q[0, h], K[0, h], V[0, h], Om, p, causal=causal)[lo:lo + lens[rank]]
            err = max(err, float(np.abs(Y[0, h].numpy() - ref).max() / np.abs(ref).max()))
        res[causal] = err
    dist.barrier()
    out.put((rank, res))
    dist.destroy_process_group()


def test_two_gloo_ranks_sequence_parallel_exchange():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_sp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, errs in res:
        assert errs[False] < 1e-9 and errs[True] < 1e-9, (rank, errs)


def test_select_states_orders_and_filters():
    a, b, c = (torch.full((2, n, 80, 256), float(i)) for i, n in enumerate((1, 2, 1)))
    sh = [torch.zeros(2, t.shape[1], 2) for t in (a, b, c)]
    g = list(zip((a, b, c), sh))
    st, s2 = sharding.select_states(g, 1, causal=False)
    assert st.shape == (2, 4, 80, 256) and s2.shape == (2, 4, 2) and st[0, :, 0, 0].tolist() == [0.0, 1.0, 1.0, 2.0]
    st, _ = sharding.select_states(g, 2, causal=True)
    assert st.shape == (2, 3, 80, 256) and st[0, :, 0, 0].tolist() == [0.0, 1.0, 1.0]
    assert sharding.select_states(g, 0, causal=True) == (None, None)
