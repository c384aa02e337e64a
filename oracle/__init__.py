"""CPU oracle for the HORA hot path.  Test infrastructure only: never imported by the product."""
