"""B200-native incremental GNN inference on evolving graphs (RIPPLE++ hot path).

`paper_2601_12347_b200.ripple` is the thin binding over the C-ABI CUDA library;
`paper_2601_12347_b200.inputs` draws the seeded synthetic inputs.  Nothing is imported eagerly so
that the input generators stay usable where the CUDA library has not been built.
"""

__all__ = ["inputs", "ripple"]
