"""B200-native DecentLaM update library: CUDA kernels behind a C ABI plus this thin binding.

    from paper_2104_11981_b200 import binding   # loads libdecentlam.so (build it first)
    from paper_2104_11981_b200 import inputs    # seeded synthetic workloads
"""
