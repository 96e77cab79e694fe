"""fp64 CPU oracle of the partitioned, micro-batched training step.  TEST INFRASTRUCTURE ONLY."""
