"""Test infrastructure only: the CPU oracle the CUDA path is checked against."""
