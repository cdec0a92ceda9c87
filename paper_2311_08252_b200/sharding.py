"""Host-side helpers for running the path on several GPUs.

Contexts (and with them every (context, head) attention unit) are independent, so the path
shards by contexts: each rank owns a contiguous slice of the global batch, holds a replica of
the datastore, and exchanges nothing on the data path.  Timing is the maximum over ranks."""
from __future__ import annotations


def shard_bounds(n_items: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of rank's contiguous slice; sizes differ by at most one, earlier ranks
    take the larger slices."""
    if world < 1 or not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(seconds: float, dist=None, device=None) -> float:
    """All-reduce(max) of a per-rank duration; identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(seconds)
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_step: int, steps: int, world: int, seconds_max: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank_step * steps * world / seconds_max


# ---------------------------------------------------------------------------------------
# A datastore spread over several GPUs: every rank holds a range of token positions with its
# own suffix array, and one decoding step's draft takes three small exchanges (winning suffix
# length, hit counts, candidate rows).  The functions below are the host logic; the compute
# steps are passed in, so the same code drives the CUDA entry points (rest_retrieve,
# rest_gather_rows, rest_draft_from_runs) and, in the CPU tests, plain stand-ins.
# ---------------------------------------------------------------------------------------
SHARD_HALO = 32          # tokens of the next shard that a shard keeps behind its own range:
                         # n_max + m <= 32 tokens follow the start of any match


def shard_tokens(tokens, rank: int, world: int, halo: int = SHARD_HALO):
    """The slice of the token stream that `rank` stores (its own position range followed by
    `halo` tokens of the next shard) and the number of positions it owns."""
    begin, end = shard_bounds(len(tokens), rank, world)
    return tokens[begin:min(len(tokens), end + halo)], end - begin


def shard_suffix_array(sa_of_slice, owned: int):
    """From the suffix array of a shard's slice to the array the shard searches: the entries
    of its own positions, order kept (works on numpy arrays and torch tensors)."""
    return sa_of_slice[sa_of_slice < owned]


class TorchComm:
    """The exchanges over torch.distributed (NCCL for CUDA tensors, gloo for CPU tensors)."""

    def __init__(self, dist, group=None):
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def all_reduce_max(self, t):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)
        return t

    def all_gather(self, t):
        """[world, ...]: every rank's tensor (same shape everywhere)."""
        import torch
        t = t.contiguous()
        out = torch.empty((self.world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out, t, group=self.group)      # rank-major concatenation
        return out.view((self.world,) + tuple(t.shape))


class ThreadComm:
    """The same exchanges between threads of one process, one thread per shard: several shards
    on one GPU (tests, or a datastore cut up to bound the suffix-array build).  All threads
    must issue their device work on the same stream."""

    def __init__(self, world: int):
        import threading
        self.world = world
        self._barrier = threading.Barrier(world)
        self._slots = [None] * world

    def view(self, rank: int):
        comm = self

        class _View:
            world = comm.world

            def __init__(self):
                self.rank = rank

            def _exchange(self, t):
                comm._slots[rank] = t
                comm._barrier.wait()
                got = list(comm._slots)
                comm._barrier.wait()
                return got

            def all_reduce_max(self, t):
                import torch
                return torch.stack(self._exchange(t)).max(dim=0).values

            def all_gather(self, t):
                import torch
                return torch.stack(self._exchange(t))

        return _View()


def allocate_rows(cnt_all, K: int):
    """How many candidate rows every shard contributes: cnt_all int64[world, B] hit counts of
    the shards that match the winning length (0 for the others).  All rows when their total is
    at most K; else shard i gets floor(K C_i / cnt) - floor(K C_(i-1) / cnt), C_i the running
    total, which sums to K and for a single shard is K."""
    import torch
    total = cnt_all.sum(dim=0, keepdim=True)
    run = torch.cumsum(cnt_all, dim=0)
    safe = torch.clamp(total, min=1)
    capped = (K * run) // safe - (K * (run - cnt_all)) // safe
    return torch.where(total <= K, cnt_all, capped)


def sharded_draft(comm, retrieve_fn, gather_fn, build_fn, ctx, ctx_len, K: int):
    """One draft over a sharded datastore.  comm: TorchComm or a ThreadComm view.
        retrieve_fn(ctx, ctx_len)                      -> match_n [B] int32, match_range [B,2] int64, status [B]
        gather_fn(match_n, match_range, take, Kr)      -> rows [B,Kr,m] int32, row_len [B,Kr] int32, status [B]
        build_fn(rows [B,R,Kr,m], row_len [B,R,Kr], run_rows [B,R], ctx_len) -> the trees
    Returns (trees, info) with info = winning length [B], total hits [B], rows taken [world,B],
    status [B] (the maximum over the shards)."""
    import torch
    match_n, match_range, status = retrieve_fn(ctx, ctx_len)
    n_star = comm.all_reduce_max(match_n.clone())
    wins = (match_n == n_star) & (n_star > 0)
    cnt = torch.where(wins, match_range[:, 1] - match_range[:, 0], torch.zeros_like(match_range[:, 0]))
    cnt_all = comm.all_gather(cnt.to(torch.int64))                     # [world, B]
    take_all = allocate_rows(cnt_all, K)
    Kr = max(1, int(take_all.max().item()))                            # row capacity of this step's runs
    take = take_all[comm.rank].to(torch.int32).contiguous()
    mine_n = torch.where(wins, match_n, torch.zeros_like(match_n))
    rows, row_len, st2 = gather_fn(mine_n, match_range, take, Kr)
    rows_all = comm.all_gather(rows)                                   # [world, B, Kr, m]
    len_all = comm.all_gather(row_len)                                 # [world, B, Kr]
    status_all = comm.all_reduce_max(torch.maximum(status, st2).clone())
    run_rows = take_all.t().contiguous().to(torch.int32)               # [B, world]
    trees = build_fn(rows_all.permute(1, 0, 2, 3).contiguous(), len_all.permute(1, 0, 2).contiguous(),
                     run_rows, ctx_len)
    return trees, {"match_n": n_star, "hits": cnt_all.sum(dim=0), "taken": take_all, "status": status_all}


def sharded_draft_cuda(comm, ds, ctx, ctx_len, n_max=16, n_min=2, K=5000, m=10, N=64, sample_mode=0):
    """sharded_draft on the CUDA entry points: `ds` is this rank's shard (a Datastore whose
    suffix array lists its own positions).  Every rank builds every tree (replicated result).
    Contexts whose shards reported a problem come back as empty trees with that status."""
    import paper_2311_08252_b200 as rest
    trees, info = sharded_draft(
        comm,
        lambda c, cl: rest.rest_retrieve(ds, c, cl, n_max=n_max, n_min=n_min),
        lambda mn, mr, take, Kr: rest.rest_gather_rows(ds, mn, mr, take, Kr, m=m, sample_mode=sample_mode),
        lambda rows, lens, runs, cl: rest.rest_draft_from_runs(rows, lens, runs, cl, m=m, N=N),
        ctx, ctx_len, K)
    import torch
    trees.status.copy_(torch.maximum(trees.status, info["status"]))
    trees.match_n.copy_(info["match_n"])
    trees.match_range[:, 0] = 0
    trees.match_range[:, 1] = info["hits"]
    return trees, info
