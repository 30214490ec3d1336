"""CPU oracle of the 8-bit training hot path.  Test infrastructure only."""
