"""CPU oracle of the draft-and-verify decision path (test infrastructure only).

Nothing in the product package imports this.  `ref` wraps the plain C fp64 oracle,
`mini` is a second, independently written NumPy fp64 statement of the same definitions
used for tiny cases and brute-force cross-checks.
"""
