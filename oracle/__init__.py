"""CPU oracle package: test infrastructure only (see moespec_oracle.py)."""
