"""B200-native FP32 GPT-2 training step (hand-written sm_100a CUDA behind a C ABI).

`paper_2606_24780_b200.binding` mirrors `include/bt.h` one to one; importing this package
does not load the CUDA library (the binding loads it on first use and fails loudly if it has
not been built: `python -m paper_2606_24780_b200.build`).
"""
__all__ = ["binding", "build"]
