"""CPU oracle of the MoE-layer hot path.  Test infrastructure only: nothing in
the product package imports it."""
