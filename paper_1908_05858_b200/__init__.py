"""B200-native binarized convolution (the hot path of daBNN, arXiv 1908.05858).

``paper_1908_05858_b200.binding`` is the thin ctypes layer over the C-ABI library
``libdabnn_b200.so`` (hand-written CUDA kernels for sm_100a); ``synth`` draws the seeded
synthetic inputs.  Nothing here falls back to the CPU: using the binding without the
compiled library raises.
"""
__all__ = ["binding", "synth", "build"]
