"""B200-native planned-arena transformer executor (layout + memory planning, sm_100a kernels).

`fluid` is the thin ctypes binding over the C-ABI library; `synth` builds the seeded synthetic
workloads. Importing this package loads nothing heavy; the CUDA library is opened on first use
and its absence is an error, never a fallback.
"""
