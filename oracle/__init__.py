"""CPU oracle of the Deep Gradient Compression hot path: test infrastructure only."""
