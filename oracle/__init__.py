"""CPU checker for the AG-gated attention layer (test infrastructure only)."""
