"""B200-native verify-and-feedback step of speculative decoding with an online-learned draft.

``paper_2603_12617_b200.binding`` wraps the C-ABI CUDA library (``include/sd_verify.h``);
``paper_2603_12617_b200.synth`` makes seeded synthetic inputs.  The CUDA library is loaded on
first use of the binding and its absence is an error: there is no CPU fallback.
"""
__all__ = ["binding", "synth", "shard"]
__version__ = "0.1.0"
