"""CPU oracle of the batched token sampler -- test infrastructure, never a product path."""
