"""CPU oracle for the EchoKV decode path (test infrastructure; see echokv_oracle.py)."""
