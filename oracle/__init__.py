"""CPU checker (test infrastructure only); see gwq_oracle.py."""
