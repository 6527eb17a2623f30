"""Host-side plumbing for running one process per GPU: which positions a rank evaluates and how
the ranks' timings are combined.  Positions are independent and the weights read-only, so the data
path itself needs no collective; only the elapsed time is reduced (maximum over ranks)."""
import torch
import torch.distributed as dist


def rank_first_index(rank: int, batch_per_rank: int) -> int:
    """Index of the first position of this rank's batch in the seeded position stream (weak scaling:
    every rank evaluates `batch_per_rank` positions of its own)."""
    return rank * batch_per_rank


def split_batch(total: int, rank: int, world: int):
    """Contiguous [begin, end) range of a `total`-position batch for this rank (strong scaling);
    the first `total % world` ranks get one position more."""
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def barrier():
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
