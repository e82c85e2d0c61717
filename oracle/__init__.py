"""CPU oracle of the GAD training epoch: test infrastructure, never imported by the CUDA library."""
