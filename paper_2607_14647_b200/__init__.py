"""B200-native verify hot path of D-cut (adaptive verification-depth pruning for batched
speculative decoding): cross-request depth selection, ragged paged verification attention
and greedy acceptance, as hand-written sm_100a kernels behind a C ABI (`libdcut.so`).

`paper_2607_14647_b200.binding` loads the library (and raises if it is not built);
`paper_2607_14647_b200.workloads` draws the seeded synthetic inputs and imports no kernel.
"""

__all__ = ["workloads"]
