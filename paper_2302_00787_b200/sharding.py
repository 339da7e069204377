"""How the path spreads over several GPUs: every (batch, head) unit is independent in all
stages, so ranks take disjoint sets of units and no data-path collective is needed.  The
only communication is the max-over-ranks of the measured time (and a barrier)."""
from __future__ import annotations

import os


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def unit_partition(n_units: int, rank: int, world: int) -> range:
    """Contiguous, disjoint, covering split of n_units (batch, head) units over `world` ranks;
    the first n_units % world ranks take one unit more."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def rank_seed(seed: int, rank: int) -> int:
    """Weak scaling: every rank runs the whole workload on its own seeded draw."""
    return seed + 7919 * rank


def max_over_ranks(value: float, backend_device=None) -> float:
    """Max of a scalar over all ranks (no-op without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, backend_device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ---------------------------------------------------------------------------------------------
# Sequence parallelism: few, long sequences.  Every rank holds a contiguous slice of the tokens of
# every (batch, head) (rank r the r-th slice).  Section 2.2's numerator and normaliser are sums over
# keys, so what the ranks exchange is the key-side sum of their slices ("key states"), never
# features: one all-gather of [B*H, ns, 80, 256] fp32 blocks per rank.  Before that, the set
# statistics of Section 4 (means over tokens) are averaged over the ranks with the slice lengths as
# weights, so that all ranks fit the same parameters.
# ---------------------------------------------------------------------------------------------
def _group_ready(group):
    import torch.distributed as dist
    return dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1


def combine_statistics(stats, n_tokens: int, group=None):
    """Token-weighted average over the ranks of per-slice statistics (every entry is a mean over tokens)."""
    import torch
    import torch.distributed as dist
    if not _group_ready(group):
        return stats
    w = torch.tensor([float(n_tokens)], dtype=torch.float64, device=stats.device)
    tot = stats * w
    dist.all_reduce(tot, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(w, op=dist.ReduceOp.SUM, group=group)
    return tot / w


def gather_key_states(state, shifts, group=None):
    """All ranks' key states, as a list indexed by rank of (state [B*H, ns_r, 80, 256], shifts [B*H, ns_r, 2]).
    Slices of equal shape on every rank (the number of pieces depends on the slice length and the device only)."""
    import torch
    import torch.distributed as dist
    if not _group_ready(group):
        return [(state, shifts)]
    world = dist.get_world_size(group)
    st = [torch.empty_like(state) for _ in range(world)]
    sh = [torch.empty_like(shifts) for _ in range(world)]
    dist.all_gather(st, state.contiguous(), group=group)
    dist.all_gather(sh, shifts.contiguous(), group=group)
    return list(zip(st, sh))


def select_states(gathered, rank: int, causal: bool):
    """The states a rank's queries see, concatenated along the piece index: all ranks' (bidirectional) or those of
    the ranks before it (causal; None when nothing precedes)."""
    import torch
    use = gathered[:rank] if causal else gathered
    if not use:
        return None, None
    return (torch.cat([s for s, _ in use], dim=1).contiguous(), torch.cat([h for _, h in use], dim=1).contiguous())


def sequence_parallel_forward(ctx, Q, K, V, Omega, variant, causal=False, qk_scale=1.0, group=None, out=None):
    """One forward pass (statistics, fit, attention) with the token axis of Q, K, V [B, H, L_local, d] spread over
    the ranks of `group` in rank order.  `ctx` provides fsharp_stats, fsharp_fit_params, fsharp_attend_key_state and
    fsharp_attend_with_state (a binding.Context).  Returns this rank's rows of Y.  Without an initialised process
    group (or with one rank) it is the single-device computation through the same calls."""
    import torch.distributed as dist
    rank = dist.get_rank(group) if _group_ready(group) else 0
    d = Q.shape[-1]
    stats = combine_statistics(ctx.fsharp_stats(Q, K, qk_scale=qk_scale), Q.shape[2], group)
    params = ctx.fsharp_fit_params(stats, d, variant)
    state, shifts = ctx.fsharp_attend_key_state(K, V, Omega, params, qk_scale=qk_scale)
    states, shs = select_states(gather_key_states(state, shifts, group), rank, causal)
    return ctx.fsharp_attend_with_state(Q, K, V, Omega, params, states, shs, causal=causal, qk_scale=qk_scale, out=out)
