"""fp64 CPU oracle of the step-attention path: test infrastructure, never the product path."""
