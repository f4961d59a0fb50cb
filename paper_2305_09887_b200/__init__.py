"""RandomTMA / SuperTMA data-parallel hot path for NVIDIA B200 (sm_100a).

``inputs`` holds the seeded synthetic-workload generators; ``binding`` is the
thin ctypes layer over the CUDA C-ABI library and is loaded on first use.
"""
