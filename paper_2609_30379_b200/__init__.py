"""libnested_pair: forward pass of a Pairformer-style block on a packed multi-ragged pair state,
hand-written CUDA for sm_100a behind a C ABI (include/nested_pair.h).  ``binding`` marshals
arguments to the shared library; ``workloads`` holds the seeded synthetic configurations."""
