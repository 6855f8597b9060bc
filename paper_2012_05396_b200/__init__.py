"""SSD-SGD (arXiv 2012.05396) update path for NVIDIA B200: Python binding of libssd_sgd.so.

Sub-modules: `binding` (the C ABI, same names), `state` (device buffers), `synth` (seeded
synthetic inputs), `build` (nvcc build of the library).  Importing the package loads nothing;
the library is loaded on first use and its absence is an error.
"""
