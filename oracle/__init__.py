"""CPU oracle of the expert-choice MoE layer.  Test infrastructure only.

Nothing under this folder is part of the product: only tests, the smoke check
and the benchmark's cpu_baseline / reference legs may import it.  It shares no
code with the CUDA path and never imports it.
"""
