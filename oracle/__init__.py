"""CPU oracle of the EAGLE-2 draft-and-verify hot path (test infrastructure, not a product path)."""
