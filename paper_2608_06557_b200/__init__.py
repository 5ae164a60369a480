"""B200-native Cascade scheduling + KV-tier step.

``paper_2608_06557_b200.cascade``  - thin binding over the C-ABI CUDA library (libcascade.so)
``paper_2608_06557_b200.workload`` - seeded synthetic input generators (numpy only)
``paper_2608_06557_b200.build``    - nvcc build of the library for sm_100a
"""
