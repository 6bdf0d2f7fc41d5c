"""Plain CPU checker for APAR tree decode attention, KV append and fork.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package: it exists
so that tests, the smoke entry and the benchmark's CPU-baseline leg have an independent,
slow and obviously correct answer to compare the CUDA library with.  It shares no code
with the CUDA path and never receives values computed by it.

* `forest`      - logical store of generation threads (no blocks, no paging).
* `attention`   - fp64 dense softmax attention over a thread's path to the root.
* `bookkeeping` - integer model of the paged pool: block tables, reference counts,
                  free list, copy-on-fork of the partial last block.
* `paragraphs`  - Algorithm 1's paragraph tree and Restore on plain token lists.

Parity status: every function here is pinned by tests under tests/ that do not go through
the function itself (library routine on a reducing special case, an independent
mask-based formulation, closed forms, hand-computed block tables).  None is "parity
unpinned".
"""
from .forest import Forest
from .attention import softmax_weights, dense_attention, tree_decode_attention
from .bookkeeping import BlockModel, BookkeepingError
from .paragraphs import SequenceGroup, FORK, CHILD, EOS

__all__ = ["Forest", "softmax_weights", "dense_attention", "tree_decode_attention",
           "BlockModel", "BookkeepingError", "SequenceGroup", "FORK", "CHILD", "EOS"]
