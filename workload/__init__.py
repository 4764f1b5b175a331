"""Seeded synthetic workloads (shapes, configurations, arrival schedules and
input generators) shared by the oracle's tests and the CUDA library's tests
and bench.  Contains none of the aggregation arithmetic."""
