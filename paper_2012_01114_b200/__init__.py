"""Skip-scheduled self-attention for B200 (sm_100a): Python front end of the C-ABI library.

`paper_2012_01114_b200.binding` loads ``libpsa.so`` (built from ``csrc/`` by
``paper_2012_01114_b200.build``) and marshals arguments; every step of the computation runs in
the library's CUDA kernels.  `paper_2012_01114_b200.inputs` draws the seeded synthetic tensors.
"""
