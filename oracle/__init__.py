"""fp64 CPU oracle for LRSA. Test infrastructure only: never imported by the CUDA package."""
