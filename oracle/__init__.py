"""CPU oracle of the time-rotated quantized linear layer: test infrastructure only."""
