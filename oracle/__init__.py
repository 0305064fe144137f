"""fp64 CPU oracle of the attention forward operator -- test infrastructure only."""
