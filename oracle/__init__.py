"""fp64 CPU oracle of the LTE layer: test infrastructure, never the product path."""
