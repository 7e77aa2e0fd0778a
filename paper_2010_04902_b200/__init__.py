"""ByzShield parameter-server aggregation on one B200: thin Python binding over libbz (C ABI).

Importing this package does not load the CUDA library; the first call into
:mod:`paper_2010_04902_b200.binding` does, and fails loudly when the library is missing.
"""

__all__ = ["binding", "inputs"]
