"""S2A 4-bit derivative stash for GELU and softmax: sm_100a CUDA kernels behind a C ABI.

``paper_2503_08154_b200.binding`` marshals torch tensors into the C-ABI calls of
``libs2a.so``; ``paper_2503_08154_b200.synth`` draws the synthetic workloads.
"""
