"""B200-native speculative-exit step (draft -> extended head -> verify -> accept -> exit).

The compute runs in ``csrc/`` (CUDA, sm_100a) behind a C ABI; ``binding`` marshals
arguments to it and ``synth`` draws the seeded synthetic inputs.  Importing the package
loads nothing; the shared library is loaded on first use and its absence is an error.
"""
