"""float64 CPU oracle of the windowed OPD divergence path: test infrastructure only."""
