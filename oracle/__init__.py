"""fp64 CPU oracle of the Sampling-VT operator -- test infrastructure only."""
