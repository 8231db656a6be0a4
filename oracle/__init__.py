"""CPU oracle of the ADSA decode-attention path (test infrastructure only)."""
