"""CPU oracle for G-CADA: test infrastructure, not part of the product path."""
