"""B200-native parameter-server update path of the Rudra framework (arXiv 1509.04210).

``binding`` wraps the C-ABI library (``include/rudra_ps.h``); ``synth`` makes seeded inputs.
The native library is loaded on first use of ``binding`` and there is no CPU fallback.
"""
