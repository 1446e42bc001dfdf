"""Float64 CPU oracle of the truncated spectral layer: test infrastructure only.

Nothing in the product path may import this package.
"""
