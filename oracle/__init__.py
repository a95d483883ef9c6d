"""CPU oracle (test infrastructure): see excp_oracle.py."""
