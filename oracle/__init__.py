"""fp64 CPU oracle for the N-way Adasum combine.  Test infrastructure only: the CUDA library and
its binding never import this package."""
