"""CPU oracle of the ETA inference path: test infrastructure, not product code."""
