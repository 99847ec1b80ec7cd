"""CPU oracle (test infrastructure only): plain reference for the CKKS linear layer."""
