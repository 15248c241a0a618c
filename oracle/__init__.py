"""CPU oracle for the batched adaptive filtered beam search -- test infrastructure only."""
