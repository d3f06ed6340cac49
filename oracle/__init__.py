"""CPU oracle of the MoE forward pass: test infrastructure, not product code."""
