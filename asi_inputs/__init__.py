"""Seeded synthetic inputs and workload tables shared by the oracle's tests and the CUDA path's tests."""
