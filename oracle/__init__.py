"""fp64 CPU oracle of the GRASS layer step: test infrastructure, never a product path."""
