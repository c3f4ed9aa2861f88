"""CPU oracle of the Hybrid Verified Decoding per-step path: test infrastructure only."""
