"""CPU oracle for the D2-MHE hot path.  TEST INFRASTRUCTURE: never imported by the CUDA library."""
