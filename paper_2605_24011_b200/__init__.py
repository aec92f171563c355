"""B200-native low-bit block-quantised linear layers (libaq).

`paper_2605_24011_b200.aq` is the binding over the C-ABI library; importing
it loads `libaq.so` and raises if the library has not been built.
`paper_2605_24011_b200.synth` holds the seeded synthetic input generators.
"""
__all__ = ["aq", "synth", "build"]
