"""Seeded synthetic workloads: combinator-program descriptions and their inputs.

This module holds data only.  It describes each benchmark program as a plain
list of node records (kind, dtype, shape, input slots, function *names*,
constant parameters) and draws the seeded input arrays.  It contains none of
the arithmetic of the combinators themselves: the CPU oracle and the CUDA
library each interpret the function names with their own tables, and neither
of them imports this module -- tests and the benchmark do, and hand the same
records and the same input arrays to both sides.
"""
from .programs import (  # noqa: F401
    Node, Program, config1, config2, config3, config4, config5,
    scatter_example, scatter_example_paper_graph, single_loop, greedy_bottom_up_bad, greedy_top_down_bad,
    simple1, simple2, simple3, simple4, simple5, segmented_sums, row_scans, suffix_sums, exclusive_scans, exclusive_row_scans, diagonal_of_product, random_program, random_int_program, random_scan_program, scan_consumers, offsets_then_gather, fold_of_scan, histogram_2d, gather_three_roots, CONFIGS,
)
from .inputs import (  # noqa: F401
    counter_bits, uniform_f32, normal_f32, uniform_int, zipf_keys, segment_offsets, make_inputs,
)
