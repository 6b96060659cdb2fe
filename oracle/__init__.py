"""CPU oracle: test infrastructure only.  Imported by tests/, the smoke check and the
benchmark's CPU-baseline leg; never by the library."""
