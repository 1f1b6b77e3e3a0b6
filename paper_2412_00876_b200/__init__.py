"""B200-native Dynamic-LLaVA sparsified-inference hot path (predictor, top-k / keep
decision, K/V compaction, attention over the compacted context).

Importing the package loads nothing; `paper_2412_00876_b200.binding` opens the CUDA
library on first use and raises if it has not been built.
"""
