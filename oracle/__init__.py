"""CPU oracle of the GraphKV compression path (test infrastructure only; see graphkv_oracle.c)."""
