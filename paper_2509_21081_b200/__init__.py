"""B200-native MLA decode attention with a shared prefix (hybrid naive/absorb).

The compute lives in ``libtyphoon_mla.so`` (CUDA, sm_100a) behind a C ABI
declared in ``include/typhoon_mla.h``; ``binding`` forwards to it one to one and
``decoder.TyphoonMLADecoder`` bundles the handle, workspace and call sequence a
user needs.  ``inputs`` draws the seeded synthetic workloads.  Importing
``binding``/``decoder`` fails loudly when the library has not been built.
"""

__all__ = ["inputs", "binding", "decoder", "build"]
