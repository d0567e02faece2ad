"""Test infrastructure: the fp64 CPU oracle of the KVM layer. Not part of the product path."""
