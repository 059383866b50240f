"""TEST INFRASTRUCTURE: the CPU oracle.  Never imported by the CUDA package."""
