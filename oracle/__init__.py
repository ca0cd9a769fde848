"""CPU oracle of the routed FP4 mixture-of-experts layer: test infrastructure, not product code."""
