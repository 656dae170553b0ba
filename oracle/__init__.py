"""CPU oracle (test infrastructure only; see tb_oracle.c and oracle.py)."""
