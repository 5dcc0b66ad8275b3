"""CPU checker for the CUDA library: test infrastructure, never imported by the product."""
