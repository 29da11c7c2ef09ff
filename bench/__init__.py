"""Measurement harness around the library (not part of the importable product package):
per-configuration report against dense cuBLAS, planner quality on the paper's grid, predictor
calibration, search loop, single-shape timing for profiler captures, seconds-long runs under the
power limit.  Run as `python -m bench.<module>` from the repository root."""
