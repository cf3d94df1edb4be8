"""CPU oracle (test infrastructure only; see gk_oracle.cpp)."""
