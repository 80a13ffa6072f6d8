"""B200-native action-conditioned decode step (attention keep-rate, MLP prune
rate and activation bit-width per sequence) behind a small C-ABI library.

`paper_2605_10875_b200.binding` loads the CUDA library and mirrors its entry
points; `paper_2605_10875_b200.synth` draws the seeded synthetic workloads.
Importing this package does not load the library.
"""
