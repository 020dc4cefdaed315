"""CPU oracle (test infrastructure only; see flowblock_oracle.py)."""
