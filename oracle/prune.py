"""Prune sets of a compiled function, written as plain definitions.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Edges (Sec. 2.2): x_i -> x_j iff some operator has x_i among its inputs and
x_j among its outputs.

Forward prune (Algorithm 1): a tensor is marked iff it is a target or a target
is reachable from it.  An operator is kept iff at least one of its outputs is
marked (Sec. 2.1: an operator with all outputs un-colored is removed).

Backward prune (Algorithm 2), for the pair set P = objs x wrts: a tensor is in
G iff it lies on some directed path wrt ~> obj (paths of length 0 count).  The
printed listing loses marks in two places (it falls through after re-marking a
node already known to connect, and it stops scanning the children of a node as
soon as one of them is the derivative target); the definition in the prose of
Sec. 2.3 ("all chains from an objective target to a derivative target") is
what is implemented here.

Two-stage DAG (Sec. 2.3): the gradient operators are unfolded after the last
forward operator.  For a stage s = (objs, wrts) the gradient operator of a
forward operator o exists iff o has an output in G and an input in G; it reads
dY for outputs Y in G (plus forward tensors through its anchor, Sec. 3.3) and
writes dX for inputs X in G.  The targets of a function are its fetched
outputs; Algorithm 1 runs over the two-stage DAG from them.  The seed d(obj)
has the objective itself as parent, so an objective of a live stage is marked.

Fed intermediates (Sec. 3.1: any tensor of the workspace can be fed by name;
Sec. 2.1: the inputs of a function are pushed in).  A tensor listed among the
inputs of a function is given, not solved: in that function's graph no edge
leads into it, so the operator that would have produced it is no parent of
it.  Every set above is then taken on the graph without those edges; a
gradient whose derivative target has lost all its chains cannot be fetched.
"""


def _children(desc):
    n = len(desc["tensors"])
    ch = [set() for _ in range(n)]
    pa = [set() for _ in range(n)]
    for op in desc["ops"]:
        for i in op["in"]:
            for o in op["out"]:
                ch[i].add(o)
                pa[o].add(i)
    return ch, pa


def _reach(start, nbrs):
    seen = set()
    stack = list(start)
    while stack:
        x = stack.pop()
        if x in seen:
            continue
        seen.add(x)
        stack.extend(nbrs[x])
    return seen


def without_edges_into(desc, fed):
    """The graph of a function whose inputs are ``fed``: every operator loses the fed tensors from its
    outputs (operator ids stay as they are; an operator left without outputs has no edge at all)."""
    fed = set(fed)
    ops = [{"type": op["type"], "in": list(op["in"]), "out": [o for o in op["out"] if o not in fed]}
           for op in desc["ops"]]
    return {"tensors": desc["tensors"], "ops": ops, "grads": desc.get("grads", [])}


def forward_marks(desc, targets):
    """Algorithm 1 as a definition: targets and everything a target is reachable from."""
    _, pa = _children(desc)
    return _reach(targets, pa)


def backward_marks(desc, objs, wrts):
    """Algorithm 2 as a definition: nodes on some path wrt ~> obj, over all pairs."""
    ch, pa = _children(desc)
    marked = set()
    for o in objs:
        anc = _reach([o], pa)
        for w in wrts:
            marked |= _reach([w], ch) & anc
    return marked


def function_sets(desc, inputs, outputs):
    """Everything the pruner decides for ``function(inputs, outputs)``.

    Returns a dict with
      marked      : list of 0/1 per tensor id (forward tensors: Algorithm 1 marks on the
                    two-stage DAG; gradient tensors: marked iff needed by a fetched target)
      fwd_ops     : kept forward operator ids, creation order (Sec. 3.2)
      grad_ops    : [(stage, forward op id, tuple of produced input positions)], stage by
                    stage, inverse creation order inside a stage (Sec. 3.2)
      used_inputs : 0/1 per listed input
    """
    desc = without_edges_into(desc, inputs)
    tensors, ops, grads = desc["tensors"], desc["ops"], desc.get("grads", [])
    n = len(tensors)
    grad_node = {}  # tensor id of a gradient tensor -> (stage, wrt)
    for s, g in enumerate(grads):
        for w, gid in zip(g["wrts"], g["grad_ids"]):
            grad_node[gid] = (s, w)

    G = [backward_marks(desc, g["objs"], g["wrts"]) for g in grads]
    for t in outputs:
        if t in grad_node:
            s, w = grad_node[t]
            if w not in G[s]:
                raise ValueError("no path from tensor %d to any objective of stage %d" % (w, s))
    producer = {}
    for k, op in enumerate(ops):
        for o in op["out"]:
            producer[o] = k

    # gradient operators of every stage and the parent relation of the two-stage DAG
    def gop_exists(s, k):
        return any(o in G[s] for o in ops[k]["out"]) and any(i in G[s] for i in ops[k]["in"])

    consumers = [[] for _ in range(n)]
    for k, op in enumerate(ops):
        for i in set(op["in"]):
            consumers[i].append(k)

    # nodes: ("f", id) forward tensors, ("g", s, id) gradient tensors
    def parents(node):
        if node[0] == "f":
            x = node[1]
            if x in grad_node:            # a gradient tensor id is an alias of its gradient node
                s, w = grad_node[x]
                return [("g", s, w)]
            if x in producer:
                return [("f", i) for i in ops[producer[x]]["in"]]
            return []
        _, s, x = node
        out = []
        if x in grads[s]["objs"]:
            out.append(("f", x))          # seed: the chain starts at the objective
        for k in consumers[x]:
            if gop_exists(s, k):
                # the forward tensors this gradient operator reads through its anchor are
                # inputs/outputs of an ancestor of the objective, so the seed edge above
                # already marks them; only the dY edges need stating
                out += [("g", s, y) for y in ops[k]["out"] if y in G[s]]
        return out

    seen = set()
    stack = [("f", t) for t in outputs]
    while stack:
        nd = stack.pop()
        if nd in seen:
            continue
        seen.add(nd)
        stack.extend(parents(nd))

    marked = [0] * n
    for nd in seen:
        if nd[0] == "f":
            marked[nd[1]] = 1
    for gid, (s, w) in grad_node.items():
        if ("g", s, w) in seen:
            marked[gid] = 1
    fwd_ops = [k for k, op in enumerate(ops) if any(marked[o] for o in op["out"])]
    grad_ops = []
    for s in range(len(grads)):
        for k in range(len(ops) - 1, -1, -1):
            if not gop_exists(s, k):
                continue
            pos = tuple(p for p, i in enumerate(ops[k]["in"])
                        if i in G[s] and ("g", s, i) in seen and i not in ops[k]["in"][:p])
            if pos:
                grad_ops.append((s, k, pos))
    used = [marked[i] for i in inputs]
    return {"marked": marked, "fwd_ops": fwd_ops, "grad_ops": grad_ops, "used_inputs": used}
