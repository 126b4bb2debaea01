"""QAM-W weight codec (encode / decode / distortion / codebook training) for NVIDIA B200.

``binding`` is the ctypes front end of the CUDA library ``libqamw.so`` (built in-tree
by ``build.build()``); ``synth`` draws the seeded synthetic benchmark inputs.
Importing the package does not load the library; the first call into ``binding`` does,
and raises if it has not been built.
"""
__all__ = ["binding", "build", "synth"]
