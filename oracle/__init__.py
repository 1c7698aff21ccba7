"""CPU oracle (test infrastructure). See litevar_oracle.py."""
