"""B200-native Muon optimizer step: thin Python binding over the C-ABI library.

Importing this package does not load the shared library; the first call into
:mod:`paper_2502_16982_b200.binding` does, and fails loudly if it is missing.
"""

__all__ = ["binding", "workloads", "build", "distributed"]
