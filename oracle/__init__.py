"""CPU oracle (test infrastructure). See cmoe_oracle.py."""
