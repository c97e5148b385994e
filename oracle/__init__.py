"""Plain, slow CPU fp64 oracle for the planned-arena transformer executor.

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke entry and by the bench's cpu-baseline
leg. The product path (the CUDA library and its Python binding) never imports, links or runs
anything in this package, and the two share no code.
"""
