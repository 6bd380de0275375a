"""Float64 CPU oracle for PaTH attention.  Test infrastructure only: nothing on
the CUDA product path imports this package."""
