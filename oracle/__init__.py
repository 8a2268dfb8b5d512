"""CPU checkers of the SparseLoCo outer step (slo), of the 12-bit position format (idx12), of the
embedding re-projection (embed) and of the activation subspace compression (subspace): test
infrastructure only, never on the product path."""
