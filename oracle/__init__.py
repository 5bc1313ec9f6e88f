"""CPU oracle for the residual-binary linear layer (test infrastructure, not product code)."""
