"""CPU oracle for the BUZZ hot path -- test infrastructure only; never imported by the product."""
