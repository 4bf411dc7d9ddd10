"""B200-native (sm_100a) UniPool MoE-layer hot path.

``synth``   seeded synthetic workloads (no method arithmetic).
``binding`` ctypes binding of the C-ABI library ``libunipool.so`` (argument
            marshalling only; every step of the path runs in CUDA kernels).

Importing the package does not load the CUDA library; ``binding.lib()`` does,
and raises if the library has not been built.
"""
