"""CPU oracle (test infrastructure only; see shadowsync_oracle.py)."""
