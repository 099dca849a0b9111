"""B200-native causal prefill partial attention (after PecSched, arXiv 2409.15104).

`binding` wraps the C-ABI library (libpec.so, built from csrc/); `workloads` holds the
seeded synthetic inputs.  There is no CPU implementation of the path in this package.
"""
