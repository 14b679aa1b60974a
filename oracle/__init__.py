"""CPU oracle for the TapOut hot path: test infrastructure, never a product dependency."""
