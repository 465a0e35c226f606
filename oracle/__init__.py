"""CPU oracle of the Kangaroo decode step: test infrastructure, never imported by the product path."""
