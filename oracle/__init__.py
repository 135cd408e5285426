"""CPU oracle of the VScan reduction path: test infrastructure only.

Nothing in the product package imports this; the CUDA library and this package
share no code.  Import sites allowed: tests, the smoke check, and the
benchmark's CPU-baseline / reference legs.
"""
