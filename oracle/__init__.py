"""CPU oracle for the PCR decode path: test infrastructure, never part of the product path."""
