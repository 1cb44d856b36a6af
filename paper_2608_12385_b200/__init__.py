"""Grouped decode step of the Decode-Branch Transformer on B200 (sm_100a).

The package is a thin binding over a C-ABI CUDA library (csrc/, include/dbt.h).  Importing
the package loads nothing; `paper_2608_12385_b200.binding` loads the shared library and
fails loudly when it has not been built.  `paper_2608_12385_b200.inputs` holds the seeded
synthetic input generators and has no dependency on the library.
"""
__all__ = ["inputs", "binding"]
