"""CPU oracle for FFF inference -- test infrastructure, never part of the product path."""
