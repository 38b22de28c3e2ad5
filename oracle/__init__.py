"""Test infrastructure: the float64 CPU oracle.  Never imported by the product package."""
