"""B200-native shared-KV attention (KV-Pipe hot path).

``paper_2608_15943_b200.kvp``   ctypes binding of the C-ABI library (loads the CUDA
                                extension; raises if it is not built)
``paper_2608_15943_b200.build`` in-tree nvcc build of that library
``paper_2608_15943_b200.synth`` seeded synthetic inputs (no arithmetic of the method)
"""
