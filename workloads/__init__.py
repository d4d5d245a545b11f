"""Seeded synthetic workloads (shapes and random tensors) shared by the CPU oracle and the
CUDA path.  Holds no arithmetic of the method."""
