"""B200-native sparse-embedding step of MTrainS-style DLRM training.

`binding` mirrors the C ABI of libmtrains_b200.so (include/mtrains_b200.h); `harness` holds the
torch plumbing (device buffers, streams) that tests, the smoke check and bench.py share;
`workload` generates the seeded synthetic inputs.  Nothing is imported eagerly so that the
input generators can be used without the CUDA library.
"""
