"""CPU oracle of the AllReduce path: test infrastructure, never a product path."""
