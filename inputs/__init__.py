"""Seeded synthetic inputs (positions, weights, workload definitions) for both the CPU oracle
and the CUDA library.  Holds none of the evaluated method's arithmetic."""
