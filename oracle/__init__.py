"""CPU oracle of the halted-prefill path: test infrastructure, not the product."""
