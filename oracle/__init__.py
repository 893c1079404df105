"""CPU oracle of the SRM decode path: test infrastructure, never imported by the product."""
