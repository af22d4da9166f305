"""TEST INFRASTRUCTURE: the CPU oracle of the EMU reshard.  Not part of the product; the CUDA path never
imports it.  Only tests, the smoke check and the benchmark's CPU-baseline / reference arm may."""
