"""CPU oracle (test infrastructure only; see ssm_oracle.py)."""
