"""NuPS sparse parameter-access path for one B200: CUDA kernels behind a C-ABI library
(``csrc/``), a thin binding (``binding.py``) and seeded synthetic inputs (``inputs.py``).

Importing the package does not load the CUDA library; ``binding.load()`` does and fails
loudly when it is missing.
"""
__all__ = ["binding", "inputs"]
