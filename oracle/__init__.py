"""CPU oracle (test infrastructure only). See goq_oracle.py."""
