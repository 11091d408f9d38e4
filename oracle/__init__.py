"""CPU oracle of the clustered-MoE layer forward.  Test infrastructure only:
nothing in the product path may import this package."""
