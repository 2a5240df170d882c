"""CPU oracle for the LC-Checkpoint hot path (test infrastructure, not part of the product)."""
