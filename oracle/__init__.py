"""CPU oracle of the GrowPage decode path: test infrastructure, never imported by the product."""
