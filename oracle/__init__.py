"""CPU oracle of the LineAR hot path — test infrastructure, never imported by the product."""
