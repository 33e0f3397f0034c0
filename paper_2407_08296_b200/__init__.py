"""B200-native Q-GaLore per-step optimizer update (hand-written sm_100a CUDA behind a C ABI).

``paper_2407_08296_b200.binding`` loads the shared library and exposes one Python function
per exported entry point; ``paper_2407_08296_b200.synth`` generates seeded synthetic inputs.
Importing the package itself loads nothing, so that the input generators stay usable on a
machine without the compiled library.
"""
__all__ = ["binding", "synth", "build"]
