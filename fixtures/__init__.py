"""Seeded input generators and bench-side rank arithmetic: shared by the tests, the smoke check and
the benchmark.  Nothing here belongs to the library, and nothing here does codec arithmetic."""
