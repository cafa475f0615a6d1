"""B200-native (sm_100a) kernels for the TwigVLM / TwigVLM++ inference hot path.

``synth`` (seeded inputs) imports without a GPU.  The binding (``twig``) loads
the compiled C-ABI library and raises if it is missing: there is no CPU
fallback for any of the calls.
"""
__all__ = ["synth"]
