"""CPU oracle for the S4R hot path: test infrastructure, never imported by the product path."""
