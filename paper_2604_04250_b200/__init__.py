"""B200-native CAWN phase accumulation (sm_100a CUDA behind a C ABI).

Importing the package is cheap and loads nothing native:

* ``paper_2604_04250_b200.binding``  ctypes binding of ``libcawn.so`` (the product path)
* ``paper_2604_04250_b200.inputs``   seeded synthetic input generators
* ``paper_2604_04250_b200.build``    compiles ``csrc/`` for sm_100a with nvcc
"""
__all__ = ["binding", "inputs", "build"]
