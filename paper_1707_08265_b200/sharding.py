"""Host logic of the multi-GPU run: one process per GPU, every rank evaluates the same compiled function on
its own slice of the leading axis, and only the tensors that are reductions over that axis are exchanged,
with one all-reduce each.  Nothing here computes on tensors: the per-shard evaluation and the all-reduce are
passed in as callables (``dragon_run`` and NCCL on the GPUs, stand-ins on CPU ranks in the tests).

Which axis, for the five workloads:
  * elementwise graphs over [N] (workloads 1-3): the element range; the gradients of broadcast scalars are
    sums over all elements -> all-reduce(sum);
  * the row DAG over [R, C] (workload 5): rows; a row sum stays inside a row, so row shards are independent;
    the gradients of the [C] row-vector inputs are column sums over all rows -> all-reduce(sum) of [C] floats;
  * the MLP (workload 4): the batch; weights and biases are replicated; the loss is a mean over the batch and
    every gradient descends from it, so a rank's results are weighted by its share of the batch and added
    -> all-reduce(sum) of loss, dW1, db1, dW2, db2 after scaling by rows_of_rank / rows.
Remote data always lands in local memory (the all-reduce's output) before any kernel reads it.
"""

LOCAL, SUM, MEAN, SAME = "local", "sum", "mean", "same"


def shard_range(n, rank, world):
    """Contiguous, balanced [lo, hi) of n elements for this rank; the shards tile [0, n)."""
    base, rem = divmod(n, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def _has_extent(desc, t, extent):
    shp = desc["tensors"][t]["shape"]
    return bool(shp) and shp[0] == extent


def shard_desc(desc, extent, new_extent):
    """The graph of one shard: every tensor whose leading extent is ``extent`` gets ``new_extent`` instead."""
    out = {"tensors": [], "ops": desc["ops"], "grads": desc.get("grads", [])}
    for t in desc["tensors"]:
        shp = list(t["shape"])
        if shp and shp[0] == extent:
            shp[0] = new_extent
        out["tensors"].append({"name": t["name"], "dtype": t["dtype"], "shape": shp})
    return out


def classify_outputs(desc, outputs, extent):
    """How every fetched tensor of a function sharded along the leading axis of length ``extent`` is put
    together from the ranks' results:
      LOCAL  it has the leading extent: every rank owns its slice, nothing is exchanged;
      SUM    a gradient without the leading extent whose objectives are sums over sharded elements:
             the ranks' results add;
      MEAN   a batch mean (SoftmaxCrossEntropy of sharded logits) or a gradient that descends from one:
             the ranks' results are weighted by their share of the axis and added;
      SAME   a forward tensor without the leading extent: the same on every rank."""
    producer = {}
    for op in desc["ops"]:
        for o in op["out"]:
            producer[o] = op
    stage_of = {}
    for st in desc.get("grads", []):
        for gid in st["grad_ids"]:
            stage_of[gid] = st

    def batch_mean(t):
        op = producer.get(t)
        return op is not None and op["type"] == "SoftmaxCrossEntropy" and _has_extent(desc, op["in"][0], extent)

    kinds = []
    for t in outputs:
        if _has_extent(desc, t, extent):
            kinds.append(LOCAL)
        elif t in stage_of:
            objs = stage_of[t]["objs"]
            if all(_has_extent(desc, o, extent) for o in objs):
                kinds.append(SUM)
            elif all(batch_mean(o) for o in objs):
                kinds.append(MEAN)
            else:
                raise ValueError("gradient tensor %d: its objectives are neither sharded tensors nor batch means" % t)
        elif batch_mean(t):
            kinds.append(MEAN)
        else:
            kinds.append(SAME)
    return kinds


def cut_feeds(desc, inputs, feeds, extent, lo, hi):
    """This rank's feeds: tensors with the leading extent are sliced, the others are passed whole."""
    return [None if f is None else (f[lo:hi] if _has_extent(desc, i, extent) else f) for i, f in zip(inputs, feeds)]


def run_sharded(evaluate_shard, summed_outputs, all_reduce, weight=None, weighted_outputs=()):
    """evaluate_shard() -> list of outputs for this rank's shard.  The outputs whose positions are listed in
    summed_outputs are partial sums and are combined with all_reduce (in place); those in weighted_outputs are
    multiplied by ``weight`` (this rank's share of the axis) first."""
    outs = evaluate_shard()
    for j in weighted_outputs:
        outs[j] *= weight
        all_reduce(outs[j])
    for j in summed_outputs:
        all_reduce(outs[j])
    return outs


def run_classified(evaluate_shard, kinds, all_reduce, share):
    """The same, driven by classify_outputs(): SUM and MEAN outputs are exchanged, MEAN ones weighted by ``share``."""
    return run_sharded(evaluate_shard, [j for j, k in enumerate(kinds) if k == SUM], all_reduce, share,
                       [j for j, k in enumerate(kinds) if k == MEAN])
