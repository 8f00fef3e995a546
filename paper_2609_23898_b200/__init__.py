"""B200-native CERAR coding pipeline (encode, ring rounds, decode) behind a C ABI.

`cerar`   thin ctypes binding of libcerar.so (argument marshalling only).
`inputs`  seeded synthetic gradient generators shaped like the paper's workloads.
`build`   compiles libcerar.so in-tree with nvcc for sm_100a.
"""
__all__ = ["cerar", "inputs", "build"]
