"""CPU oracle of the OQM path: test infrastructure, never imported by the CUDA package."""
