"""CPU oracle of the SubGen streaming attention data structure.

Test infrastructure only: tests, the smoke check and the benchmark's CPU-baseline
leg may import this package. The CUDA library never does, and nothing here imports
the CUDA library or its binding.
"""
