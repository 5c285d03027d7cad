"""Float64 CPU oracle of the dAD / rank-dAD per-layer path -- test infrastructure only."""
