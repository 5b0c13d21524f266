"""B200-native draft-tree generation and greedy verification for the combined
token/embedding speculator (arXiv 2404.19124, Sec. 3.1 / Sec. 4.1).

`synth` (seeded inputs) is import-light; the CUDA binding is loaded on first use of
`paper_2404_19124_b200.binding` and fails loudly when the compiled library is missing.
"""
__all__ = ["synth", "binding"]
