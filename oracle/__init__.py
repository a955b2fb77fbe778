"""CPU oracle of the FastMKA path: test infrastructure, never imported by the product package."""
