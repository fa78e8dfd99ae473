"""CPU oracle (test infrastructure).  Not importable from the product path."""
