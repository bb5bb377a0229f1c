"""fp64 CPU oracle of the OSSCAR per-layer solve: test infrastructure, never used by the CUDA path."""
