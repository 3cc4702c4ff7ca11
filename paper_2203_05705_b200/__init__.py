"""B200-native hot path of Approximate Random Dropout (arXiv 2203.05705).

`paper_2203_05705_b200.ard` is the thin binding over the C-ABI library
(`libard.so`, built in-tree by `paper_2203_05705_b200.build`).  Importing this
package does not load the library; the first call into `ard` does, and raises
if the library is missing -- there is no CPU fallback.
"""
__all__ = ["ard", "inputs", "build"]
