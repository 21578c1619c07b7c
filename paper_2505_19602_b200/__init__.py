"""ScaleKV per-scale hot path for B200 (sm_100a): ctypes binding over the C-ABI library."""
