"""Seeded synthetic workloads (layer shapes, bitwidth draws, integer codes). No method arithmetic."""
