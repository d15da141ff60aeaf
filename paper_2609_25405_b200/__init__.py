"""B200-native mixed-batch transformer step (decode rows + embedding chunks +
incremental pooling) behind a C-ABI CUDA library.

`paper_2609_25405_b200.binding` loads the library and raises if it is missing;
there is no CPU fallback.  `paper_2609_25405_b200.synth` only generates seeded
inputs and is importable without the library.
"""
