"""CPU oracle of the H-Spec draft step: test infrastructure, never on the product path."""
