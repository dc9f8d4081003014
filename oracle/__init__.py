"""CPU oracle (fp64, plain numpy).  Test infrastructure: not part of the product path."""
