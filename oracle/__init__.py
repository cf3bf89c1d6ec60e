"""CPU oracle of the BATQuant W4A4 path: test infrastructure, never imported by the product."""
