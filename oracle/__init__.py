"""Float64 CPU oracle of the LCKV decode path.  Test infrastructure only."""
