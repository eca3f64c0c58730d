"""B200-native memory-slice hot path: slice arena allocator, per-layer prefetch of lent KV
blocks into a staging ring, paged GQA decode attention over the prepared addresses, and reclaim
migration. Everything runs in the CUDA library ``libemaslice.so``; this package only marshals
arguments (``binding``) and draws synthetic inputs (``synth``)."""
