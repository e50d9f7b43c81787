"""B200-native budgeted-KV decode attention (BaKlaVa, arXiv 2502.13176).

`binding` wraps the C-ABI library (`libbaklava.so`, built from `csrc/`); `synth`
and `workloads` produce the seeded synthetic inputs.  Importing the package does
not load the library; the first call into `binding` does, and raises if it is
missing: there is no fallback path.
"""
