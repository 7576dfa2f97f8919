"""Barrier-free symmetric-memory AllReduce for one B200 (emulated ranks).

``paper_2607_16100_b200.symar``  -- ctypes binding of the C-ABI library
``paper_2607_16100_b200.synth``  -- seeded synthetic inputs (no arithmetic of the method)
``paper_2607_16100_b200.build``  -- nvcc build of the library for sm_100a
"""
