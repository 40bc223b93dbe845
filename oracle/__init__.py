"""CPU oracle of the method -- test infrastructure, never imported by the CUDA package."""
