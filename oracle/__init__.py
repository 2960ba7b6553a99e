"""fp64 CPU oracle of the ASI hot path -- test infrastructure, never imported by the product package."""
