"""B200-native W4A4 WUSH linear layer (arXiv 2512.00956): Python binding package.

`paper_2512_00956_b200.wush` wraps the C-ABI library `libwush.so` (built from
`csrc/`); `paper_2512_00956_b200.synth` generates the seeded synthetic inputs.
Importing the package does not load the library; the first call into `wush` does,
and raises if it has not been built.
"""
__all__ = ["synth", "wush"]
