"""B200 (sm_100a) fused attention forward: O = softmax(scale * Q K^T [+ causal mask]) V with LSE.

`api` binds the C ABI of libattn_fwd.so; `inputs` holds the seeded synthetic input recipes;
`build` compiles the library in-tree.  Submodules are imported on demand so that the input
generator can be used without loading the CUDA library.
"""
