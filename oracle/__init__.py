"""Float64 CPU oracle.  Test infrastructure only: imported by tests/, by the
smoke check and by the benchmark's CPU-baseline leg, never by the product."""
