"""FB4 online activation quantizer for B200 (sm_100a): Python binding of the C-ABI library.

`paper_2603_02883_b200.fb4` is the binding (argument marshalling only; every step of
the path runs in the CUDA kernels of csrc/); `paper_2603_02883_b200.synth` makes the
seeded synthetic inputs.  Importing the package itself loads nothing.
"""
