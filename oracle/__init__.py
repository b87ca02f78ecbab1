"""Test infrastructure: the fp64 CPU oracle.  Not part of the product package."""
