"""CPU oracle of the FreeBalance hot path: test infrastructure, never imported by the product."""
