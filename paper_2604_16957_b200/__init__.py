"""B200-native fused int4 compressed-domain decode attention.

`paper_2604_16957_b200.tq`      -- thin ctypes binding of the C-ABI CUDA library (libtq.so)
`paper_2604_16957_b200.inputs`  -- seeded synthetic workloads (numpy only, no arithmetic of the method)
`paper_2604_16957_b200.build`   -- nvcc build of the library for sm_100a
"""
