"""CPU oracle of the exponent-reuse codec.  Test infrastructure only."""
