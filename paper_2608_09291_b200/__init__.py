"""B200-native W4A4 bitmap-sparse SpMM (IE-BME weights x dense INT4 activations).

``workloads`` holds the seeded input generators; ``binding`` is the ctypes front end of the
C-ABI library built from ``csrc/`` (import it explicitly: it needs the compiled library).
"""
