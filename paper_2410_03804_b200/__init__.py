"""B200-native hot path of the Mixture-of-Attentions drafter (arXiv 2410.03804).

`moa` holds the ctypes binding over the C-ABI library (csrc/, built by `build`);
`synth` holds the seeded synthetic input generators. Importing the package loads
neither the library nor CUDA; `moa.load_library()` does.
"""
__all__ = ["moa", "synth", "build"]
