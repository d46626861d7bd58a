"""CPU oracle for the NVFP4 path: test infrastructure only, never imported by the product."""
