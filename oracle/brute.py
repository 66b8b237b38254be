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
