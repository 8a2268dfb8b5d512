"""CPU checker of the SparseLoCo outer step: test infrastructure only."""
