"""CPU oracle of the MoTE FFN-layer forward pass.  Test infrastructure only: nothing in the
product path may import this package."""
