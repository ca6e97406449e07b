"""B200-native ABS (adaptive bounded staleness) parameter-server round loop.

`paper_2301_08895_b200.abs` is the binding of the C-ABI library built from
`csrc/`; `paper_2301_08895_b200.inputs` holds the synthetic input generators.
Importing the package does not load the CUDA library; the first call does, and
fails loudly if the library has not been built.
"""
