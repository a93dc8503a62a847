"""Seeded synthetic inputs and network shapes shared by the oracle's tests and the CUDA library's tests and benchmark."""
