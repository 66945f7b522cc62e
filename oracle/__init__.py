"""CPU oracle of the block-sparse operator (test infrastructure, independent of the CUDA path)."""
