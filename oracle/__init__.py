"""CPU oracle for Linnea-equation evaluation.  TEST INFRASTRUCTURE ONLY.

`oracle.plan`   -- exhaustive (Catalan) parenthesization with property-aware multiplication counts.
`oracle.values` -- fp64 dense left-to-right evaluation built on a C triple loop.

Nothing in the CUDA library imports, links or executes anything in this package, and this package
imports nothing from the library.  Allowed users: the test-suite, the smoke check, and the
benchmark's CPU-baseline / reference legs.
"""
