"""CPU oracle of the HERO cached step: test infrastructure, never imported by the product path."""
