"""fp64 CPU oracle for paged decode attention: test infrastructure, never on the product path."""
