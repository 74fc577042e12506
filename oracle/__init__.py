"""CPU oracle of the SDVG hot path.  Test infrastructure: never imported by the product."""
