"""CPU oracle of the split speculative verification round.  Test infrastructure only."""
