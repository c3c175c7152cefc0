"""CPU oracle package: test infrastructure only (see snapstream_oracle.py)."""
