"""B200-native chunk-wise KV-cache codec and tolerance score (LLMS, arXiv 2403.11805).

`binding` wraps the C-ABI library (csrc/ -> libllms.so); `synth` makes the seeded
synthetic inputs.  Importing the package loads nothing; the library is loaded on
the first call into `binding`, and a missing library is an error, never a fallback.
"""
