"""CPU oracle (test infrastructure).  See worldkv_oracle.py."""
