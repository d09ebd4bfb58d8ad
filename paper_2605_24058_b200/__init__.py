"""B200-native LoRDBA adapter forward: y += s_out * (B_sign (s_r * (A_sign (s_in * x)))).

``workloads`` (seeded synthetic inputs) imports without a GPU; the CUDA binding
is loaded on first use of ``paper_2605_24058_b200.lordba``.
"""
__version__ = "0.1.0"
