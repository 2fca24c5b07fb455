"""CPU oracle of the melded FP8-LoRA layer: test infrastructure, never a product path.

Only tests/, the smoke check and the benchmark's CPU-baseline leg import this.
"""
