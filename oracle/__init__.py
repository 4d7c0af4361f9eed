"""CPU oracle of the FEPLB MoE-layer hot path (test infrastructure; see feplb_oracle)."""
