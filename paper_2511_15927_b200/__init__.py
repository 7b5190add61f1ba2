"""B200-native bidirectional Mamba-2 mixer (DiffuMamba denoising step): C-ABI CUDA library + thin binding.

`paper_2511_15927_b200.inputs` draws seeded synthetic inputs and needs no GPU; the binding in
`paper_2511_15927_b200.binding` loads the compiled library and raises if it is missing.
"""
