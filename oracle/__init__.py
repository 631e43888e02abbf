"""CPU oracle for Y = act(A.B + bias): test infrastructure, never on the product path."""
