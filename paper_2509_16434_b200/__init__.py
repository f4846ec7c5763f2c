"""B200-native PPO learner step over an on-device rollout buffer of depth frames.

The CUDA library is loaded on first use of `paper_2509_16434_b200.binding`; importing
the package (or `synth`, the input generators) loads nothing native.
"""
__all__ = ["synth", "binding"]
