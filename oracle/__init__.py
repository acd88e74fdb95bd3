"""CPU fp64 oracle (test infrastructure; see tree_oracle.py).  Never imported by the product package."""
