"""B200-native hot path of C-Coll (arXiv 2304.03890): error-bounded compression of fp32 collective buffers,
its decoder, the fused decompress-add-recompress ring round, and single-GPU replays of C-Allreduce and
C-Bcast / C-Scatter.  The product is csrc/ (CUDA kernels + C ABI, built into libccoll.so); binding.py
marshals arguments; fields.py makes seeded synthetic inputs.
"""
