"""fp64 CPU oracle for ConvBN Eval / Deploy / Tune mode.  Test infrastructure only: the CUDA
library and its binding never import this package."""
