"""B200-native batch verifier for register-allocation candidates.

The package has two halves that never import each other's internals:

* ``synth``   -- seeded synthetic programs and candidate rows (inputs only, no
                 verification arithmetic).
* ``binding`` -- ctypes marshalling onto the C ABI of ``libverilocc.so`` (the CUDA
                 library under ``csrc/``).  Importing it fails loudly when the
                 library has not been built; there is no CPU fallback.

Nothing is imported eagerly here so that ``synth`` stays usable on machines
without the CUDA library.
"""

__all__ = ["synth", "binding", "build"]
