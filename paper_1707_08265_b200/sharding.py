"""Host logic of the multi-GPU run of an elementwise function: every rank owns a contiguous
shard of the element range and evaluates the same compiled function on it; tensors that are
sums over all elements (gradients of broadcast scalars) are the only exchange, one all-reduce.
Nothing here computes on tensors; the per-shard evaluation is passed in as a callable."""


def shard_range(n, rank, world):
    """Contiguous, balanced [lo, hi) of n elements for this rank; the shards tile [0, n)."""
    base, rem = divmod(n, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def run_sharded(evaluate_shard, summed_outputs, all_reduce):
    """evaluate_shard() -> list of outputs for this rank's shard; the outputs whose positions are
    listed in summed_outputs are partial sums and are combined with all_reduce (in place)."""
    outs = evaluate_shard()
    for j in summed_outputs:
        all_reduce(outs[j])
    return outs
