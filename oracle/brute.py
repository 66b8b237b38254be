"""Brute-force prune sets by enumerating every simple directed path (exponential).

TEST INFRASTRUCTURE ONLY.  Independent of oracle/prune.py: no reachability
sets, no memo -- each path is walked edge by edge.  Usable only on tiny DAGs.
"""


def _edges(desc):
    e = set()
    for op in desc["ops"]:
        for i in op["in"]:
            for o in op["out"]:
                e.add((i, o))
    return sorted(e)


def all_paths(desc):
    """Every directed path (as a tuple of tensor ids), including the single-node paths."""
    n = len(desc["tensors"])
    edges = _edges(desc)
    out = []

    def extend(path):
        out.append(tuple(path))
        for (a, b) in edges:
            if a == path[-1]:
                extend(path + [b])

    for x in range(n):
        extend([x])
    return out


def forward_marks_bruteforce(desc, targets):
    """Sec. 2.2: nodes that can affect a target = nodes on a path that ends in a target."""
    m = set()
    for p in all_paths(desc):
        if p[-1] in targets:
            m.update(p)
    return m


def backward_marks_bruteforce(desc, objs, wrts):
    """Sec. 2.3: nodes on a chain between an objective and a derivative target, all pairs."""
    m = set()
    for p in all_paths(desc):
        if p[0] in wrts and p[-1] in objs:
            m.update(p)
    return m


# ---- the two-stage DAG of Sec. 2.3, written out node by node -----------------------------------

def two_stage_dag(desc):
    """Nodes and edges (parent -> child) of the DAG in which every gradient operator is unfolded behind
    the last forward one.  Nodes: ("f", x) for every forward tensor, ("g", s, x) for every stage s and
    every tensor x on a chain wrt ~> obj of that stage (found by path enumeration).  Edges:
      * forward operators: every input to every output (Sec. 2.2);
      * the gradient operator of forward operator k in stage s exists iff k has an output and an input
        on a chain; it reads dY for its outputs Y on a chain and writes dX for its inputs X on a chain:
        an edge ("g",s,Y) -> ("g",s,X) for every such pair;
      * through its anchor (Sec. 3.3) it also reads the forward tensors of its Run-Op: an edge from
        every input of k, and from every output of k that is on a chain, to every dX it writes;
      * the chain of stage s starts at the objective itself: ("f", obj) -> ("g", s, obj).
    """
    grads = desc.get("grads", [])
    edges = set()
    for op in desc["ops"]:
        for i in op["in"]:
            for o in op["out"]:
                edges.add((("f", i), ("f", o)))
    for s, st in enumerate(grads):
        G = backward_marks_bruteforce(desc, set(st["objs"]), set(st["wrts"]))
        for o in st["objs"]:
            if o in G:
                edges.add((("f", o), ("g", s, o)))
        for op in desc["ops"]:
            ys = [y for y in op["out"] if y in G]
            xs = [x for x in op["in"] if x in G]
            if not ys or not xs:
                continue
            for x in xs:
                for y in ys:
                    edges.add((("g", s, y), ("g", s, x)))
                for t in list(op["in"]) + ys:
                    edges.add((("f", t), ("g", s, x)))
    return edges


def function_sets_bruteforce(desc, inputs, outputs):
    """What function(inputs, outputs) keeps, from the definition alone: a node of the two-stage DAG is
    marked iff it lies on some path that ends in a fetched node (Algorithm 1 as prose: "can affect a
    target").  Every path is walked edge by edge, no reachability sets.  Same result layout as
    oracle.prune.function_sets.  A listed input is given (Sec. 3.1: fed by name), so the operator that
    would have produced it loses it as an output: no edge of the function's graph ends in it."""
    given = set(inputs)
    desc = {"tensors": desc["tensors"], "grads": desc.get("grads", []),
            "ops": [dict(op, out=[y for y in op["out"] if y not in given]) for op in desc["ops"]]}
    tensors, ops, grads = desc["tensors"], desc["ops"], desc.get("grads", [])
    edges = sorted(two_stage_dag(desc))
    alias = {}
    for s, st in enumerate(grads):
        for w, gid in zip(st["wrts"], st["grad_ids"]):
            alias[gid] = ("g", s, w)
    targets = {alias.get(t, ("f", t)) for t in outputs}
    marked_nodes = set()

    def walk_up(path):              # extend the path backwards, parent by parent
        marked_nodes.update(path)
        for (a, b) in edges:
            if b == path[0]:
                walk_up([a] + path)

    for t in targets:
        walk_up([t])
    n = len(tensors)
    marked = [0] * n
    for t in range(n):
        if t in alias:
            marked[t] = int(alias[t] in marked_nodes)
        else:
            marked[t] = int(("f", t) in marked_nodes)
    fwd_ops = [k for k, op in enumerate(ops) if any(marked[o] for o in op["out"])]
    grad_ops = []
    for s, st in enumerate(grads):
        G = backward_marks_bruteforce(desc, set(st["objs"]), set(st["wrts"]))
        for k in range(len(ops) - 1, -1, -1):
            op = ops[k]
            if not (any(y in G for y in op["out"]) and any(x in G for x in op["in"])):
                continue
            pos = tuple(p for p, x in enumerate(op["in"])
                        if x in G and ("g", s, x) in marked_nodes and x not in op["in"][:p])
            if pos:
                grad_ops.append((s, k, pos))
    return {"marked": marked, "fwd_ops": fwd_ops, "grad_ops": grad_ops, "used_inputs": [marked[i] for i in inputs]}
