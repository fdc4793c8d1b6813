"""relay-race GR inference on one B200: C-ABI CUDA library plus a thin Python binding.

``binding`` mirrors the C entry points one to one; ``runtime`` owns device memory
(through PyTorch) for callers that want objects instead of raw pointers; ``synth``
draws the seeded synthetic inputs.  Nothing here computes: every step of the path
runs in the CUDA library, and importing ``binding`` fails loudly without it.
"""
