"""B200 (sm_100a) implementation of the {-1,+1} bit-plane decomposed quantized layer.

``paper_2106_09886_b200.qnn``       -- thin ctypes binding of the C-ABI library ``libqnn.so``
                                      (importing it fails loudly when the library is not built).
``paper_2106_09886_b200.workloads`` -- seeded synthetic inputs (no arithmetic of the method).
``paper_2106_09886_b200.build``     -- compiles ``csrc/*.cu`` with nvcc for sm_100a.
"""
__version__ = "0.1.0"
