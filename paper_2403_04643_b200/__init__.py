"""QAQ (arXiv 2403.04643) hot path for B200: C-ABI CUDA library `libqaq.so` + ctypes binding.

`paper_2403_04643_b200.qaq`    the binding (same names as include/qaq.h)
`paper_2403_04643_b200.synth`  seeded synthetic inputs
`paper_2403_04643_b200.build`  in-tree nvcc build of the library
"""
