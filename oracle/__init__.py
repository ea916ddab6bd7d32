"""Test infrastructure only: the double-precision CPU oracle.  Never imported by the product path."""
