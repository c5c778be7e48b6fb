"""CPU oracle for combinator programs.  TEST INFRASTRUCTURE, not a product path.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It shares no code with the CUDA library and never calls
it; the CUDA library never calls it either.

  interp        node-at-a-time interpreter, every array materialised (numpy;
                fp64 accumulation for fp32 folds, scans and scatters)
  cluster_loop  the loop a fused cluster denotes, in pure Python (small sizes)
  legality      the paper's legality model evaluated for a given clustering,
                and the enumeration of every legal clustering
  functions     the element-level function tables

Pins (see tests/test_oracle_*.py): hand-worked examples per combinator, closed
forms, the equivalences and the printed loops of the paper, the printed graph
and clusterings of `scatterExample`, agreement of the two evaluators over every
legal clustering.  Not pinned by anything but its own definition: the exact
stream of the Zipf sampler in the input generator (only its range and its
leading frequency are checked) -- "parity unpinned" for that generator, which
is an input recipe and not part of the method.
"""
from . import functions, interp, legality, cluster_loop  # noqa: F401
