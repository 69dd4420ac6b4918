"""CPU oracle (test infrastructure).  See qcfg_oracle.py."""
