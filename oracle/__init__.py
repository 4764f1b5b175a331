"""CPU oracle of the model-aggregation hot path.  TEST INFRASTRUCTURE ONLY:
nothing in the product package may import it."""
