"""MixLoRA feed-forward block (arXiv 2404.15159) for NVIDIA B200: thin binding over the C-ABI library.

The CUDA library does all the work; this package only marshals arguments.  Importing
`paper_2404_15159_b200.binding` fails loudly when the built library is missing.
"""
