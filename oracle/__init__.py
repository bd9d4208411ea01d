"""CPU oracle for the BSR fine-tuning step: test infrastructure, never on the product path."""
