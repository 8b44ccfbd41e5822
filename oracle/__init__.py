"""CPU oracle (test infrastructure only).  See revffn_oracle.py."""
