"""CPU oracle of the bounded-state restore path (test infrastructure, never on the product path)."""
