"""B200-native hot path of SpecVLM's pruned-draft speculative decoding step.

``synth`` (input generators) imports without the CUDA library; ``specvlm`` (the binding)
loads ``libspecvlm.so`` on first use and fails loudly when it is missing.
"""
__all__ = ["synth", "specvlm"]
