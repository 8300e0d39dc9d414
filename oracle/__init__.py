"""CPU oracle of the biased-local-SGD hot path: test infrastructure only."""
