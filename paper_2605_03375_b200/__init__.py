"""B200-native KV-cache object-store hot path: per-layer restore / save between
contiguous KV objects and a paged KV pool, with GPU-built submission descriptors.

`workload` holds the seeded input generators; `tutti` is the thin binding over the
C-ABI CUDA library (imported lazily so that the generators work without it)."""
