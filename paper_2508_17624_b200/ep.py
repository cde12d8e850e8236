"""Expert parallelism for the adapter-aware MoE layer (Section 5.1: tensor parallelism for self-attention, expert
parallelism for the MoE layers; Section 5.2 runs TP = EP = 8 and TP = EP = 2).

Placement.  Rank r of R holds the base experts `owned_range(M, R, r)` together with every adapter's re-tuned copies
of them, and the shared experts `owned_range(S, R, r)`.  A (token, expert) pair is computed where its *base* expert
lives: rerouting through the expert map replaces a base expert by an adapter's copy of that same expert, so it never
moves a pair to another rank.  The virtual weight tensors and the expert map are identical on all ranks; only the
slots a rank owns are backed by physical pages there.

Exchange.  The paper does not describe one.  Under tensor-parallel attention every rank already holds the hidden
states of all tokens, so no token travels: every rank routes all tokens (the router is replicated), computes the
pairs whose expert it holds, and the ranks' fp32 partial sums are added by one all-reduce per layer; the sum is
rounded to bf16 once.  All arithmetic of a rank runs in the library (`ew_moe_forward_partial`, `ew_ep_finish`);
this module only places the all-reduce (torch.distributed: NCCL on GPUs) between the two calls.
"""
from typing import Optional, Tuple


def owned_range(n: int, size: int, rank: int) -> Tuple[int, int]:
    """[lo, hi) of n items held by `rank` of `size`: contiguous blocks of ceil(n / size), the last ones short or
    empty.  The library computes the same ranges from ep_size / ep_rank."""
    size = max(int(size), 1)
    per = -(-n // size)
    lo = min(n, rank * per)
    return lo, min(n, lo + per)


def owner_of(j: int, n: int, size: int) -> int:
    """Rank that holds item j of n."""
    size = max(int(size), 1)
    return j // (-(-n // size))


def local_pair_mask(topk_ids, num_experts: int, size: int, rank: int):
    """Boolean mask over the [B, k] router choices (base expert ids): the pairs rank `rank` computes."""
    lo, hi = owned_range(num_experts, size, rank)
    return (topk_ids >= lo) & (topk_ids < hi)


class ExpertParallelLayer:
    """One rank's side of an expert-parallel forward.

    `pool`: a `binding.Pool` created with ep_size = world size and ep_rank = this process's rank (anything with
    `moe_forward_partial(layer, x, adapter_ids)` and `ep_finish(summed)` will do: the CPU tests pass a stand-in).
    `group`: the torch.distributed process group of the R ranks (None: the default group; with no process group
    initialised the layer runs as a single rank).
    """

    def __init__(self, pool, group=None):
        self.pool = pool
        self.group = group

    def world(self) -> int:
        import torch.distributed as dist
        if not (dist.is_available() and dist.is_initialized()):
            return 1
        return dist.get_world_size(self.group)

    def forward(self, layer: int, x, adapter_ids, out: Optional[object] = None):
        """x: [B, H] bf16 (the same on every rank), adapter_ids: [B] int32 -> [B, H] bf16 (the same on every rank)."""
        partial = self.pool.moe_forward_partial(layer, x, adapter_ids)
        if self.world() > 1:
            import torch.distributed as dist
            # the layer's one exchange step: fp32 sum over ranks (stream-ordered after the partial forward)
            dist.all_reduce(partial, op=dist.ReduceOp.SUM, group=self.group)
        if out is None:
            return self.pool.ep_finish(partial)
        return self.pool.ep_finish(partial, out)
