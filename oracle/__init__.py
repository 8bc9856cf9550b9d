"""CPU oracle (test infrastructure only; see loqt_oracle.py)."""
