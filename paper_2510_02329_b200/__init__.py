"""B200-native verification step for judge speculative decoding (C-ABI library + thin binding).

``synth`` (input generators) imports without the CUDA library; everything in ``binding``
loads ``libsjverify.so`` on first use and raises if it is missing.
"""
