"""CPU oracle for the ANPD draft-and-verify path: test infrastructure only.

Nothing in the CUDA library or its Python binding imports this package; only
tests/, the smoke check and the benchmark's CPU-baseline leg do."""
