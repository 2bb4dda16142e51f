"""CPU oracle for BitLinear (test infrastructure only; never imported by the product path)."""
