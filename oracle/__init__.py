"""CPU oracle for the A^3 fusion hot path: test infrastructure, never imported by the product path."""
