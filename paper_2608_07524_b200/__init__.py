"""B200-native packed variable-length attention (forward and backward) and the single-GPU
micro-batch planner, behind a C ABI.  ``inputs`` holds the seeded synthetic workloads;
``binding`` is the ctypes layer over ``libdcp.so`` (loaded on first use)."""
