"""CPU oracle for the VQ linear layer: test infrastructure, never imported by the product path."""
