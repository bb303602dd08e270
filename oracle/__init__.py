"""fp64 CPU oracle of the FVAttn hot path.  Test infrastructure: never imported by the product."""
