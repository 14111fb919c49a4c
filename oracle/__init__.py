"""XFP oracle package: test infrastructure only (tests/, the smoke check and the benchmark's
CPU-baseline leg).  The product package never imports it."""
