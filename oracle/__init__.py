"""CPU oracle package: test infrastructure only.  Nothing on the product path imports it."""
