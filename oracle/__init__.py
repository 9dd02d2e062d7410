"""CPU oracle of the verifier path: test infrastructure, never imported by the product."""
