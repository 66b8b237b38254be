"""The interpreter run over independent chunks of the leading axis, on a pool of worker processes.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Nothing of the method changes here: an elementwise graph treats every element alike, and in a
row-reduction graph Sum and Mean stay inside a row, so a function over [N] or [R, C] tensors can be
evaluated on slices of the leading axis one after the other (or side by side) with
oracle.interp.run_function unchanged.  Tensors that do not have the leading extent (row vectors,
scalars) are fed whole to every chunk.  A fetched tensor without the leading extent is a sum over
that axis when it is a gradient (of a broadcast operand, Sec. 2.3: contributions add; the reverse sweep
is linear in the upstream gradient, so the per-chunk results are added in fp64) and is the same in every
chunk when it is a forward tensor.  Fetched tensors with the leading extent are either returned, or compared on the
spot with values handed in (so that a full-size comparison never holds more than a chunk per worker).

The pool is started with the "spawn" method: a forked child of a process that has already
initialised CUDA hangs.
"""
import multiprocessing as mp
import os

import numpy as np

from . import interp


def with_leading_extent(desc, old, new):
    """The same graph with every tensor's leading extent ``old`` replaced by ``new``."""
    out = {"tensors": [], "ops": desc["ops"], "grads": desc.get("grads", [])}
    for t in desc["tensors"]:
        shp = list(t["shape"])
        if shp and shp[0] == old:
            shp[0] = new
        out["tensors"].append({"name": t["name"], "dtype": t["dtype"], "shape": shp})
    return out


def _chunk(args):
    desc, extent, lo, hi, inputs, outputs, feeds, compare, tol, dtype, with_floor = args
    d = with_leading_extent(desc, extent, hi - lo)
    res = interp.run_function(d, inputs, outputs, feeds, dtype=np.dtype(dtype).type)
    low = interp.run_function(d, inputs, outputs, feeds, dtype=np.float32) if with_floor else None
    out = []
    grad_ids = {gid for st in desc.get("grads", []) for gid in st["grad_ids"]}
    for k, (o, r) in enumerate(zip(outputs, res)):
        shp = desc["tensors"][o]["shape"]
        if not (shp and shp[0] == extent):
            # a gradient of a broadcast operand: this chunk's share of the sum; a forward tensor: the same in every chunk
            out.append(("sum" if o in grad_ids else "same", np.asarray(r, dtype=np.float64)))
        elif compare is not None and compare[k] is not None:
            got = np.asarray(compare[k], dtype=np.float64)
            err = np.abs(got - r) / (tol * (1 + np.abs(r)))
            err = np.where(np.isfinite(err), err, np.inf)
            j = int(np.argmax(err)) if err.size else 0
            floor = 0.0
            if low is not None:     # the same arithmetic in fp32 on the CPU against fp64, in tolerances
                fe = np.abs(low[k].astype(np.float64) - r) / (tol * (1 + np.abs(r)))
                floor = float(np.max(np.where(np.isfinite(fe), fe, np.inf))) if fe.size else 0.0
            out.append(("err", float(err.reshape(-1)[j]) if err.size else 0.0, lo, j,
                        float(got.reshape(-1)[j]) if err.size else 0.0, float(np.asarray(r).reshape(-1)[j]) if err.size else 0.0, floor))
        else:
            out.append(("val", np.asarray(r)))
    return out


def default_workers():
    return max(1, min(os.cpu_count() or 1, 32))


def run_chunked(desc, inputs, outputs, feeds, extent, chunk, workers=None, compare=None, tol=1e-5, dtype="float64", pool=None,
                with_floor=False):
    """Evaluates function(inputs, outputs) over chunks [lo, lo + chunk) of the leading axis of length
    ``extent``.  feeds: arrays in the order of inputs (None for a pruned input).  compare: optional list,
    per output an array of the output's full shape (or None) to compare against chunk by chunk.

    Returns a list per output: ("sum", array) for a tensor without the leading extent, ("err", worst
    normalised error, chunk start, flat index inside the chunk, got, ref, floor) where compare was given,
    else ("val", array of the full shape).  floor (with_floor): the worst normalised distance, over the
    whole tensor, between this interpreter run in float32 and in float64: how far fp32 rounding alone
    moves the result of this graph on these inputs."""
    workers = workers or default_workers()
    for st in desc.get("grads", []):      # a sum over chunks needs objectives that are themselves cut into chunks
        for o in st["objs"]:
            shp = desc["tensors"][o]["shape"]
            assert shp and shp[0] == extent, "objective %d does not have the leading extent" % o
    n_tasks = (extent + chunk - 1) // chunk

    def tasks():      # cut lazily: the pool's feeder blocks on its pipe, so only a few chunks exist at a time
        for lo in range(0, extent, chunk):
            hi = min(extent, lo + chunk)

            def cut(i, a):
                if a is None:
                    return None
                shp = desc["tensors"][i]["shape"]
                return np.ascontiguousarray(a[lo:hi]) if (shp and shp[0] == extent) else a

            fc = [cut(i, a) for i, a in zip(inputs, feeds)]
            cc = None if compare is None else [None if c is None else cut(o, c) for o, c in zip(outputs, compare)]
            yield (desc, extent, lo, hi, inputs, outputs, fc, cc, tol, dtype, with_floor)

    own = pool is None and workers > 1 and n_tasks > 1
    if own:
        pool = mp.get_context("spawn").Pool(workers)
    try:
        parts = list(pool.imap(_chunk, tasks())) if pool is not None else [_chunk(t) for t in tasks()]
    finally:
        if own:
            pool.close()
            pool.join()
    res = []
    for k in range(len(outputs)):
        kind = parts[0][k][0]
        if kind == "sum":
            tot = parts[0][k][1].copy()
            for p in parts[1:]:
                tot = tot + p[k][1]
            res.append(("sum", tot))
        elif kind == "same":
            res.append(("sum", parts[0][k][1]))
        elif kind == "err":
            worst = max((p[k] for p in parts), key=lambda e: e[1])
            res.append(worst[:6] + (max(p[k][6] for p in parts),))
        else:
            res.append(("val", np.concatenate([p[k][1] for p in parts], axis=0)))
    return res
