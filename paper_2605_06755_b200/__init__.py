"""GXPO active-phase parameter update for NVIDIA B200 (sm_100a).

The compute path is the CUDA shared library `libgxpo.so` built from `csrc/`;
`binding` is a thin ctypes layer over its C ABI (include/gxpo.h).  There is no
CPU fallback: importing `binding` without the built library raises.
"""
