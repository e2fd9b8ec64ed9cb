"""CPU oracle of the PQ-HSA decode operator: test infrastructure, never on the product path."""
