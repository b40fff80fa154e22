"""fp64 CPU oracle of the Block-attention hot path.  Test infrastructure only."""
