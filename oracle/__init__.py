"""CPU oracle (test infrastructure only; see solon_oracle.py)."""
