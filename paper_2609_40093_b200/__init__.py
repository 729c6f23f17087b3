"""B200-native routing-aware expert-parallel token dispatch and combine.

`paper_2609_40093_b200.ep` is the Python binding of the C-ABI CUDA library
(argument marshalling only); `paper_2609_40093_b200.inputs` draws the seeded
synthetic workloads. Importing this package loads nothing: the CUDA library is
opened on the first call of a binding function and a missing library is an error.
"""
__all__ = ["ep", "inputs"]
