"""Q-GenX reference oracle (test infrastructure only; never imported by the product path)."""
