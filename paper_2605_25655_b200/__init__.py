"""B200 (sm_100a) FP16 Llama-style decoder forward: prefill and decode.

`paper_2605_25655_b200.thinfer` is the ctypes binding over the C-ABI library
(`include/thinfer.h`); `paper_2605_25655_b200.synth` draws the seeded synthetic
inputs.  Importing the package loads neither torch nor the shared library.
"""
