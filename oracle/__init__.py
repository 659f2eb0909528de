"""CPU checker package (test infrastructure only; see bpc_oracle)."""
