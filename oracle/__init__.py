"""CPU oracle (test infrastructure).  Never import this from the product package."""
