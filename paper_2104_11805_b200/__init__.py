"""B200-native sparse-DNN SGD hot path (forward, backward, masked update) behind a C ABI.

`binding` wraps libsdnn.so one-to-one; `build` compiles it.  Importing this package does not
load the library; the first call does, and raises if it has not been built.
"""
from .binding import (  # noqa: F401
    SdnnError, Sdnn, load_library, exported_symbols, infer_noalloc, infer_noalloc_bad_columns, NOALLOC_MAX_TILE_FLOATS, probe_gather_rate, probe_gather_inflight, probe_layer_boundary, probe_smem_gather_rate, probe_word_rate, probe_tma_gather_rate, probe_mixed_gather, cluster_layer, FLAG_REORDER, FLAG_SMEM_WINDOWS, FLAG_IDX32,
    FLAG_BWD_ATOMICS, FLAG_BWD_CSC, FLAG_KEEP_DEBUG, FLAG_SKIP_DEAD, FLAG_NO_GRAPH, FLAG_NO_PDL, FLAG_BWD_ONE_LAUNCH, FLAG_ONE_TILE, ACT_CLAMPED_RELU, ACT_SIGMOID,
)
