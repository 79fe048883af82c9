"""B200-native (sm_100a) hot path of streamlined few-bit QNN inference.

Few-bit integer GEMM WwAa (w, a <= 4; unsigned, signed, bipolar) fused with the
per-output-channel multi-threshold activation, fed by packed channel-interleaved
im2col, behind a C ABI (``include/qnn.h``).  ``binding`` exposes the C entry
points under the same names; ``synth`` draws the seeded synthetic inputs.

Importing the package does not load the CUDA library; ``binding`` does, and it
raises if the library has not been built -- there is no CPU fallback.
"""

__all__ = ["binding", "synth", "build"]
