"""B200-native blockwise verification for trajectory-level speculative decoding
of diffusion language models: a thin binding over the ``libtsd`` C-ABI library
(hand-written sm_100a kernels).  There is no CPU fallback: every operation
raises if the CUDA library is missing."""
