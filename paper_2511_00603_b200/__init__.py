"""B200-native categorized serving step (EPARA's BS + MT + MF on one GPU).

`paper_2511_00603_b200.epara` is the binding over the C-ABI library; `synth` holds the seeded
workload generators.  Importing the package does not load the CUDA library.
"""
