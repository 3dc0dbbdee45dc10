"""CPU oracle of the MEPIC hot path: test infrastructure, never part of the product path."""
