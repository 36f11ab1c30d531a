"""B200-native Sentinel verifier check (arXiv 2603.03592): C-ABI library + Python binding.

``binding`` loads ``libsentinel.so`` (hand-written sm_100a kernels behind a C ABI) and mirrors
its entry points; ``synth`` draws seeded synthetic stage-boundary traffic; ``replicas`` holds
the host-side logic for running independent replicas on several GPUs.
"""
__all__ = ["binding", "synth", "replicas"]
