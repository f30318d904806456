"""CPU oracle for the WUSH-KV hot path: test infrastructure, never imported by the product path."""
