"""CPU oracle of the compression hot path (test infrastructure, never used by the product)."""
