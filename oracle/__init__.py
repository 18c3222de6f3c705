"""CPU checkers for the SPAR-K decode path.  Test infrastructure only."""
