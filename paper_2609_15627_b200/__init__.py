"""B200-native routed mixture-of-experts layer with FP4 expert weights.

`moe` is the thin binding over the C-ABI CUDA library (argument marshalling only);
`inputs` draws the seeded synthetic workloads.  Importing the package does not load
the CUDA library; the first call into `moe` does, and fails loudly if it is missing.
"""
