"""Measurement and test harness of the repack library: seeded workload generators
(``workloads``), device-resident problems on top of the C-ABI binding (``device``), the ctypes
binding of the harness kernels -- pool fill, whole-pool verifier, decode-read proxy --
(``kernels``, built from ``csrc/harness.cu`` into ``libvtoken_harness.so``), and the
one-process-per-GPU plumbing of the benchmark (``parallel``).

Nothing here is part of the repack path: the product is ``paper_2608_13263_b200`` (kernels and
binding).  Importing this package loads no native library; ``workloads`` needs numpy only.
"""
