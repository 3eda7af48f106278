"""CPU oracle (test infrastructure only).  See ``oracle.talon_oracle``."""
