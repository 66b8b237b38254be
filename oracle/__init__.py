"""CPU oracle for the Dragon graph-VM hot path (arXiv 1707.08265).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, node-at-a-time fp64
restatement of what a compiled ``function(inputs, outputs)`` (Sec. 2.1) computes
after the forward prune (Sec. 2.2, Algorithm 1) and the backward prune
(Sec. 2.3, Algorithm 2), plus the in-place structures of the pruned graph
(Sec. 2.4, Algorithm 3; oracle/inplace.py, pinned in tests/test_inplace.py by
the definition written out on tiny DAGs).  It shares no code with the CUDA library, imports
nothing from it, and must never be reached from the product path.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may use it.

Graph description consumed by every function here (a plain dict):

    {"tensors": [{"name": str, "dtype": "f32"|"bf16"|"i32", "shape": [..]}, ...],
     "ops":     [{"type": str, "in": [tensor ids], "out": [tensor ids]}, ...],
     "grads":   [{"objs": [ids], "wrts": [ids], "grad_ids": [ids]}, ...]}

Tensor and operator ids are positions in these lists, i.e. creation order
(Sec. 3.2: available operators keep their creating order).  ``grad_ids[j]`` is
the id of the tensor that holds d(sum of all elements of all objs)/d(wrts[j]).

Pins (see tests/test_oracle_*.py): brute-force path enumeration on tiny DAGs,
the paper's y = a*x example (b must stay unmarked), closed-form derivatives of
x*sin(a*x+b), central finite differences, library cross-checks for InnerProduct
and SoftmaxCrossEntropy.  Values of one specific random DAG (the two random-DAG
workloads) are pinned only through the per-operator pins plus composition.
"""
