"""CPU oracle of the mixed-precision step.  Test infrastructure only."""
