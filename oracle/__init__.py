"""fp64 CPU oracle of the token-tree verification step: test infrastructure only."""
