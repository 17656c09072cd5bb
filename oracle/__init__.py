"""CPU fp64 oracle of the DART token-reduction step: test infrastructure only.

Nothing in the product package may import this; see ``dart_oracle.c`` for the arithmetic.
"""
from .dart_oracle import (OracleResult, build, compact, gather_rows, pivots, reduce, retention,  # noqa: F401
                          retention_any, retention_global, retention_union, scores, similarity, similarity_any, splitmix64,
                          pivots_mixed, pivots_random)
