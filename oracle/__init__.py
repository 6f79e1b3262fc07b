"""CPU oracle of the SCOPE layer: test infrastructure, never part of the product path."""
