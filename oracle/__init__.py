"""CPU oracle for the ETR MoE layer: test infrastructure only (see etr_oracle.hpp)."""
