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
rounded to bf16 once.  All arithmetic of a rank runs in the library; this module only places the exchange between the
library's calls.  Three forms of it:

  forward           ew_moe_forward_partial -> all-reduce (torch.distributed; NCCL on GPUs) -> ew_ep_finish
  forward_gathered  ew_moe_forward_partial -> all-gather -> ew_ep_finish_gathered: the partial sums are added in rank
                    order on every rank, so the result has the same bits everywhere and in every run
  forward_scatter   ew_moe_forward_scatter -> barrier -> ew_ep_finish_gathered: the combine kernel itself stores the
                    partial sums into every rank's gather buffer over peer memory (no collective call on the data path);
                    the caller supplies the peer-visible buffers and the barrier (e.g. from symmetric memory)
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

    def forward_gathered(self, layer: int, x, adapter_ids, out: Optional[object] = None):
        """Same result up to the order of the fp32 additions, but deterministic: every rank adds the R partial sums in
        rank order."""
        import torch
        partial = self.pool.moe_forward_partial(layer, x, adapter_ids)
        world = self.world()
        gathered = torch.empty((world,) + tuple(partial.shape), dtype=partial.dtype, device=partial.device)
        if world > 1:
            import torch.distributed as dist
            dist.all_gather(list(gathered.unbind(0)), partial, group=self.group)     # block r = rank r's partial sums
        else:
            gathered[0].copy_(partial)
        if out is None:
            return self.pool.ep_finish_gathered(gathered)
        return self.pool.ep_finish_gathered(gathered, out)

    def forward_scatter(self, layer: int, x, adapter_ids, gather_ptrs, my_gather_buf, barrier, out: Optional[object] = None):
        """The exchange inside the combine kernel.  `gather_ptrs`: device int64 tensor with the addresses of all ranks'
        gather buffers (fp32 [R, B, H] each, peer-visible), `my_gather_buf`: this rank's own buffer as a tensor,
        `barrier`: a callable that returns once every rank's scatter for this step has completed, ordered on the current
        stream (with torch's symmetric memory: the handle's barrier).  Not exercised on more than one GPU in this
        repository's tests; on one GPU the ranks are pools on the same device and the barrier is stream order."""
        self.pool.moe_forward_scatter(layer, x, adapter_ids, gather_ptrs)
        barrier()
        if out is None:
            return self.pool.ep_finish_gathered(my_gather_buf)
        return self.pool.ep_finish_gathered(my_gather_buf, out)
