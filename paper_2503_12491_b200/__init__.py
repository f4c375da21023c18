"""B200-native CAKE prefill-time KV-cache eviction (arXiv 2503.12491).

`binding` wraps the C-ABI of libcake.so (hand-written CUDA for sm_100a);
`synth` generates the seeded synthetic workloads; `harness` glues the two for
tests and benchmarks.  Nothing in this package computes the method on the CPU.
"""
from .binding import Cake, CakeError, load_library, LIB_PATH  # noqa: F401
