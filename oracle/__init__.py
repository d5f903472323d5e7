"""CPU checker for the tests (fp64, numpy). Test infrastructure only: never on the product path."""
