"""B200-native adjoint-method gradients for a diagonal selective SSM layer.

The product is the C-ABI library built from ``csrc/`` (see ``include/adjoint_ssm.h``);
``binding`` is a thin ctypes layer over it and ``synth`` holds the seeded input recipes.
Importing the package does not load the library; the first call through ``binding`` does,
and raises if the library has not been built.
"""

__all__ = ["binding", "synth", "build"]
