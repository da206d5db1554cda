"""CPU oracle of the RanDeS superpose / retrieve path (test infrastructure only)."""
