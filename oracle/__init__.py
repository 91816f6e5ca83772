"""fp64 CPU oracle of the MoDSE layer.  Test infrastructure only: nothing in the
CUDA product path imports this package."""
