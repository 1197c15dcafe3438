"""CPU oracle for Superposed Decoding: test infrastructure, never on the product path."""
