"""fp64 CPU oracle of the DeaMoE layer -- TEST INFRASTRUCTURE.

Imported only by tests, the smoke check and the benchmark's cpu_baseline leg.
The CUDA library neither imports nor links anything from here.
"""
