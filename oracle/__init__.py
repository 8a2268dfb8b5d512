"""CPU checkers of the SparseLoCo outer step (slo), of the 12-bit position format (idx12) and of the
embedding re-projection (embed): test infrastructure only, never on the product path."""
