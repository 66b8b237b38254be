"""In-place structures of a pruned graph (Sec. 2.4, Algorithm 3).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The rule of Sec. 2.4: an in-place structure is a path of nodes that each have at most one child;
given an ancestor, the longest such path from it is found and every node on it may be renamed to
the ancestor (it may share the ancestor's memory).  Algorithm 3 visits the nodes in graph order
and, from each node not yet renamed, walks forward while the current node has exactly one child.
The graph is the pruned one (the paper renames after pruning, since renaming makes the graph
cyclic): only marked tensors and kept operators take part.

rename_dictionary() follows the algorithm's steps; rename_dictionary_bruteforce() is the
definition written out with no shared state: RD[x] is the first node a, in graph order, whose
forward single-child walk passes through x.
"""


def _children(desc, marked, kept_ops):
    ch = {x: [] for x in marked}
    for k in kept_ops:
        op = desc["ops"][k]
        for i in op["in"]:
            if i not in ch:
                continue
            for o in op["out"]:
                if o in ch and o not in ch[i]:
                    ch[i].append(o)
    return ch


def rename_dictionary(desc, marked, kept_ops):
    """Algorithm 3: {tensor: ancestor} over the marked tensors, ancestors tried in graph (creation) order."""
    ch = _children(desc, set(marked), kept_ops)
    rd = {}
    for start in sorted(ch):
        x = start
        while x not in rd:              # DepthFirstSearch(x, ancestor = start), written as a loop
            rd[x] = start
            if len(ch[x]) != 1:
                break
            x = ch[x][0]
    return rd


def rename_dictionary_bruteforce(desc, marked, kept_ops):
    """For every x the smallest a whose walk a -> only child -> only child ... reaches x."""
    ch = _children(desc, set(marked), kept_ops)
    rd = {}
    for x in ch:
        for a in sorted(ch):
            walk, y = [a], a
            while len(ch[y]) == 1 and ch[y][0] not in walk:
                y = ch[y][0]
                walk.append(y)
            if x in walk:
                rd[x] = a
                break
    return rd
