"""B200-native per-layer candidate sweep of the Scaled Outer Product PTQ method.

The package holds three things and nothing else:

* ``inputs``   -- seeded synthetic layers and the codebook ("atom") alphabets.  Pure data: it
                  contains none of the method's arithmetic and is the only module that both the
                  CUDA path and the CPU oracle's tests draw from.
* ``binding``  -- ctypes marshalling for the C-ABI library built from ``csrc/`` (``libsop.so``).
                  Every step of the sweep runs in the library's CUDA kernels; the binding only
                  converts arguments.  It raises if the library is missing: there is no CPU fallback.
* ``csrc``     -- the sm_100a CUDA kernels and the ``extern "C"`` boundary declared in ``include/sop.h``.

Nothing is imported eagerly so that ``paper_2605_14929_b200.inputs`` can be used on a machine that
has neither a GPU nor the built library.
"""

__all__ = ["inputs", "binding", "pipeline"]
