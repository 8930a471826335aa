"""CPU fp64 oracle (test infrastructure only; never on the product path)."""
