"""B200-native L4Q linear layer: forward, backward and low-bit export.

The compute lives in the CUDA library ``libl4q.so`` (see ``include/l4q.h``);
``paper_2402_04902_b200.binding`` is the thin ctypes layer over its C ABI and
``paper_2402_04902_b200.synth`` draws the seeded synthetic workloads.
Importing the package does not load the library; the first call into
``binding`` does, and raises if the library is missing.
"""
